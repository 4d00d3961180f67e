"""ctypes binding of libqnn.so: same names as the C ABI (include/qnn.h), torch tensors in and out.

Argument marshalling only -- every step runs inside the library's CUDA kernels.  The
library must have been built (``python -m paper_2106_09886_b200.build``); importing this
module without it raises ImportError, and there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libqnn.so"

OK, E_ARG, E_ALIGN, E_RANGE, E_SCALE, E_CUDA, E_DEVICE = 0, -1, -2, -3, -4, -5, -6
RELU = 1
W_NTC, W_TCN, W_NCT = 0, 1, 2

EXPORTS = [
    "qnn_status_string", "qnn_version", "qnn_row_words", "qnn_planes_bytes", "qnn_weights_bytes",
    "qnn_weights_row_words", "qnn_encode_pack", "qnn_pack_weights", "qnn_bgemm", "qnn_bconv2d",
    "qnn_bgemm_encode", "qnn_bconv2d_encode", "qnn_bconv2d_general", "qnn_mbit_encoder_forward",
    "qnn_mbit_encoder_backward", "qnn_bgemm_backward_data_workspace", "qnn_bgemm_backward_data",
    "qnn_bgemm_backward_weights_workspace", "qnn_bgemm_backward_weights", "qnn_bconv2d_backward_data_workspace",
    "qnn_bconv2d_backward_data", "qnn_bconv2d_backward_weights_workspace", "qnn_bconv2d_backward_weights", "qnn_unpack_codes_f32",
    "qnn_tensor_path_status", "qnn_last_device_status", "qnn_selftest_bounded_wait", "qnn_bgemm_int8_tensor_workspace", "qnn_bgemm_int8_tensor",
    "qnn_absmax_f32", "qnn_fc_forward_host", "qnn_fc_forward_host_pipelined", "qnn_fc_forward_noalloc", "qnn_probe_bitops", "qnn_probe_naive_sgemm", "qnn_probe_copy", "qnn_popcounts_per_output",
]
NOALLOC_SCRATCH_BYTES = 8 << 20


class QnnError(RuntimeError):
    def __init__(self, status: int, call: str):
        self.status = status
        super().__init__(f"{call} failed: {status_string(status)} ({status})")


def _load() -> C.CDLL:
    if not _LIB_PATH.exists():
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2106_09886_b200.build` "
                          "(there is no fallback path)")
    lib = C.CDLL(str(_LIB_PATH))
    p, i, i64, f, u, sz = C.c_void_p, C.c_int, C.c_int64, C.c_float, C.c_uint, C.c_size_t
    lib.qnn_status_string.restype = C.c_char_p
    lib.qnn_status_string.argtypes = [i]
    lib.qnn_version.restype = i
    lib.qnn_row_words.restype = sz
    lib.qnn_row_words.argtypes = [i64]
    lib.qnn_planes_bytes.restype = sz
    lib.qnn_planes_bytes.argtypes = [i64, i64, i]
    lib.qnn_weights_bytes.restype = sz
    lib.qnn_weights_bytes.argtypes = [i, i, i, i]
    lib.qnn_weights_row_words.restype = sz
    lib.qnn_weights_row_words.argtypes = [i, i]
    lib.qnn_encode_pack.argtypes = [p, i64, i, i64, i, f, u, p, p, p]
    lib.qnn_pack_weights.argtypes = [p, i, i, i, i, i, f, p, p]
    lib.qnn_bgemm.argtypes = [p, i, p, i, i64, i, i, f, p, i64, p, p]
    lib.qnn_bconv2d.argtypes = [p, i, p, i] + [i] * 9 + [f, p, p, p]
    lib.qnn_bconv2d_general.argtypes = [p, i, p, i] + [i] * 12 + [f, p, p, p]
    lib.qnn_bgemm_encode.argtypes = [p, i, p, i, i64, i, i, f, p, p, i, f, u, p, p, i64, p]
    lib.qnn_bconv2d_encode.argtypes = [p, i, p, i] + [i] * 9 + [f, p, p, i, f, u, p, p, p]
    lib.qnn_mbit_encoder_forward.argtypes = [p, sz, i, f, p, p]
    lib.qnn_mbit_encoder_backward.argtypes = [p, p, sz, i, f, p, p]
    lib.qnn_bgemm_backward_data_workspace.restype = sz
    lib.qnn_bgemm_backward_data_workspace.argtypes = [sz, sz, sz]
    lib.qnn_bgemm_backward_data.argtypes = [p, p, sz, sz, sz, i, f, p, i, f, p, p, sz, p]
    lib.qnn_bgemm_backward_weights_workspace.restype = sz
    lib.qnn_bgemm_backward_weights_workspace.argtypes = [sz, sz, sz]
    lib.qnn_bgemm_backward_weights.argtypes = [p, p, sz, sz, sz, i, f, p, p, sz, p]
    lib.qnn_unpack_codes_f32.argtypes = [p, sz, sz, i, i, p, sz, p]
    lib.qnn_bconv2d_backward_data_workspace.restype = sz
    lib.qnn_bconv2d_backward_data_workspace.argtypes = [i] * 9
    lib.qnn_bconv2d_backward_data.argtypes = [p, p, i] + [i] * 9 + [f, p, i, f, p, p, sz, p]
    lib.qnn_bconv2d_backward_weights_workspace.restype = sz
    lib.qnn_bconv2d_backward_weights_workspace.argtypes = [i] * 9
    lib.qnn_bconv2d_backward_weights.argtypes = [p, p, i] + [i] * 9 + [f, p, p, sz, p]
    lib.qnn_tensor_path_status.argtypes = [C.POINTER(C.c_uint)]
    lib.qnn_last_device_status.argtypes = [C.POINTER(C.c_uint)]
    lib.qnn_selftest_bounded_wait.argtypes = [u, p]
    lib.qnn_popcounts_per_output.restype = i64
    lib.qnn_popcounts_per_output.argtypes = [i] * 7
    lib.qnn_bgemm_int8_tensor_workspace.restype = sz
    lib.qnn_bgemm_int8_tensor_workspace.argtypes = [i64, i, i]
    lib.qnn_bgemm_int8_tensor.argtypes = [p, i, p, i, i64, i, i, f, p, p, p, sz, p]
    lib.qnn_absmax_f32.argtypes = [p, sz, p, p]
    lib.qnn_fc_forward_host.argtypes = [p, i64, i, i, f, u, p, i, i, f, p, p, p, p, p]
    lib.qnn_fc_forward_host_pipelined.argtypes = [p, i64, i, i, f, u, p, i, i, f, p, p, p, p, i64, C.POINTER(C.c_void_p), i]
    lib.qnn_fc_forward_noalloc.argtypes = [p, i64, i, i64, i, f, u, p, i, i, f, p, i64, p]
    lib.qnn_probe_bitops.argtypes = [i, i, i, p, C.POINTER(C.c_double), p]
    lib.qnn_probe_copy.argtypes = [p, p, sz, p]
    lib.qnn_probe_naive_sgemm.argtypes = [p, p, p, i, i, i, p]
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.qnn_status_string(int(status)).decode()


def version() -> int:
    return int(lib.qnn_version())


def row_words(k: int) -> int:
    return int(lib.qnn_row_words(k))


def planes_bytes(rows: int, k: int, bits: int) -> int:
    return int(lib.qnn_planes_bytes(rows, k, bits))


def weights_bytes(n_out: int, taps: int, c_in: int, bits: int) -> int:
    return int(lib.qnn_weights_bytes(n_out, taps, c_in, bits))


def weights_row_words(taps: int, c_in: int) -> int:
    return int(lib.qnn_weights_row_words(taps, c_in))


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _check(rc: int, call: str):
    if rc != OK:
        raise QnnError(rc, call)


def _dev(t: torch.Tensor, dtype, name: str):
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if t.dtype != dtype or not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous {dtype}")
    return t


def encode_pack(x: torch.Tensor, bits: int, scale: float, flags: int = 0, planes: torch.Tensor | None = None,
                rowsum: torch.Tensor | None = None, k: int | None = None, stream=None) -> torch.Tensor:
    """x fp32 [rows, ldx] (first k columns used) -> planes int32-typed storage [rows, bits, row_words(k)]."""
    _dev(x, torch.float32, "x")
    rows, ldx = x.shape[0] if x.dim() == 2 else x.numel() // x.shape[-1], x.shape[-1]
    k = ldx if k is None else k
    if planes is None:
        planes = torch.empty((rows, bits, row_words(k)), dtype=torch.int32, device=x.device)
    _check(lib.qnn_encode_pack(_ptr(x), rows, k, ldx, bits, float(scale), flags, _ptr(planes), _ptr(rowsum),
                               _stream(stream)), "qnn_encode_pack")
    return planes


def pack_weights(w: torch.Tensor, n_out: int, taps: int, c_in: int, layout: int, bits: int, scale: float,
                 packed: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Real weights (any of the W_* layouts, n_out*taps*c_in elements) -> packed blob (uint8 tensor)."""
    _dev(w, torch.float32, "w")
    if w.numel() != n_out * taps * c_in:
        raise ValueError("w has the wrong number of elements")
    if packed is None:
        packed = torch.empty(weights_bytes(n_out, taps, c_in, bits), dtype=torch.uint8, device=w.device)
    _check(lib.qnn_pack_weights(_ptr(w), n_out, taps, c_in, layout, bits, float(scale), _ptr(packed),
                                _stream(stream)), "qnn_pack_weights")
    return packed


def bgemm(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, Mg: int, Ng: int, Kg: int,
          alpha: float, out: torch.Tensor | None = None, acc: torch.Tensor | None = None, want_acc: bool = False,
          stream=None):
    if out is None:
        out = torch.empty((Mg, Ng), dtype=torch.float32, device=a_planes.device)
    if acc is None and want_acc:
        acc = torch.empty((Mg, Ng), dtype=torch.int32, device=a_planes.device)
    _check(lib.qnn_bgemm(_ptr(a_planes), ab, _ptr(w_packed), wb, Mg, Ng, Kg, float(alpha), _ptr(out),
                         out.stride(0), _ptr(acc), _stream(stream)), "qnn_bgemm")
    return (out, acc) if (want_acc or acc is not None) else out


def conv_out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return (size + 2 * pad - k) // stride + 1


def bconv2d(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, N: int, H: int, W: int, Cin: int,
            Cout: int, R: int, S: int, stride: int, pad: int, alpha: float, out: torch.Tensor | None = None,
            acc: torch.Tensor | None = None, want_acc: bool = False, stream=None):
    Ho, Wo = conv_out_dim(H, R, stride, pad), conv_out_dim(W, S, stride, pad)
    if out is None:
        out = torch.empty((N, Ho, Wo, Cout), dtype=torch.float32, device=a_planes.device)
    if acc is None and want_acc:
        acc = torch.empty((N, Ho, Wo, Cout), dtype=torch.int32, device=a_planes.device)
    _check(lib.qnn_bconv2d(_ptr(a_planes), ab, _ptr(w_packed), wb, N, H, W, Cin, Cout, R, S, stride, pad,
                           float(alpha), _ptr(out), _ptr(acc), _stream(stream)), "qnn_bconv2d")
    return (out, acc) if (want_acc or acc is not None) else out


def conv_general_out_dim(size: int, k: int, stride: int, pad: int, dilation: int = 1, transposed: bool = False,
                         out_pad: int = 0) -> int:
    if not transposed:
        return (size + 2 * pad - dilation * (k - 1) - 1) // stride + 1
    return (size - 1) * stride - 2 * pad + dilation * (k - 1) + 1 + out_pad


def bconv2d_general(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, N: int, H: int, W: int, Cin: int,
                    Cout: int, R: int, S: int, stride: int, pad: int, dilation: int, transposed: bool, out_pad: int,
                    alpha: float, out: torch.Tensor | None = None, acc: torch.Tensor | None = None,
                    want_acc: bool = False, stream=None):
    """Dilated or transposed convolution; out [N, Ho, Wo, Cout] with the output size of the chosen form."""
    Ho = conv_general_out_dim(H, R, stride, pad, dilation, transposed, out_pad)
    Wo = conv_general_out_dim(W, S, stride, pad, dilation, transposed, out_pad)
    if out is None:
        out = torch.empty((N, Ho, Wo, Cout), dtype=torch.float32, device=a_planes.device)
    if acc is None and want_acc:
        acc = torch.empty((N, Ho, Wo, Cout), dtype=torch.int32, device=a_planes.device)
    _check(lib.qnn_bconv2d_general(_ptr(a_planes), ab, _ptr(w_packed), wb, N, H, W, Cin, Cout, R, S, stride, pad,
                                   dilation, int(transposed), out_pad, float(alpha), _ptr(out), _ptr(acc),
                                   _stream(stream)), "qnn_bconv2d_general")
    return (out, acc) if (want_acc or acc is not None) else out


def bgemm_encode(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, Mg: int, Ng: int, Kg: int, alpha: float,
                 next_bits: int, next_scale: float, next_flags: int = 0, next_planes: torch.Tensor | None = None,
                 out: torch.Tensor | None = None, ch_gamma: torch.Tensor | None = None,
                 ch_beta: torch.Tensor | None = None, encode: bool = True, stream=None):
    """FC layer whose epilogue applies an optional per-feature affine and (encode=True) the next layer's encoder.
    Returns the next layer's activation planes, or `out` when encode is False."""
    if encode and next_planes is None:
        next_planes = torch.empty((Mg, next_bits, row_words(Ng)), dtype=torch.int32, device=a_planes.device)
    _check(lib.qnn_bgemm_encode(_ptr(a_planes), ab, _ptr(w_packed), wb, Mg, Ng, Kg, float(alpha), _ptr(ch_gamma),
                                _ptr(ch_beta), next_bits, float(next_scale), next_flags,
                                _ptr(next_planes) if encode else None, _ptr(out),
                                out.stride(0) if out is not None else Ng, _stream(stream)), "qnn_bgemm_encode")
    return next_planes if encode else out


def bconv2d_encode(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, N: int, H: int, W: int, Cin: int,
                   Cout: int, R: int, S: int, stride: int, pad: int, alpha: float, next_bits: int, next_scale: float,
                   next_flags: int = 0, next_planes: torch.Tensor | None = None, out: torch.Tensor | None = None,
                   ch_gamma: torch.Tensor | None = None, ch_beta: torch.Tensor | None = None, encode: bool = True,
                   stream=None):
    """Convolution whose epilogue applies an optional per-feature affine and (encode=True) the next layer's
    encoder: returns planes [N*Ho*Wo, next_bits, row_words(Cout)], or `out` when encode is False."""
    Ho, Wo = conv_out_dim(H, R, stride, pad), conv_out_dim(W, S, stride, pad)
    if encode and next_planes is None:
        next_planes = torch.empty((N * Ho * Wo, next_bits, row_words(Cout)), dtype=torch.int32, device=a_planes.device)
    _check(lib.qnn_bconv2d_encode(_ptr(a_planes), ab, _ptr(w_packed), wb, N, H, W, Cin, Cout, R, S, stride, pad,
                                  float(alpha), _ptr(ch_gamma), _ptr(ch_beta), next_bits, float(next_scale), next_flags,
                                  _ptr(next_planes) if encode else None, _ptr(out), _stream(stream)),
           "qnn_bconv2d_encode")
    return next_planes if encode else out


def mbit_encoder_forward(x: torch.Tensor, bits: int, r: float = 1.0, c: torch.Tensor | None = None, stream=None):
    """Eq. 10: c fp32 [bits, n] with c[m-1] = phi^m(x / r) in {-1, 0, +1}."""
    _dev(x, torch.float32, "x")
    if c is None:
        c = torch.empty((bits, x.numel()), dtype=torch.float32, device=x.device)
    _check(lib.qnn_mbit_encoder_forward(_ptr(x), x.numel(), bits, float(r), _ptr(c), _stream(stream)),
           "qnn_mbit_encoder_forward")
    return c


def mbit_encoder_backward(x: torch.Tensor, gc: torch.Tensor, bits: int, r: float = 1.0, gx: torch.Tensor | None = None,
                          stream=None):
    """Eq. 12: gradient with respect to x given the gradients gc [bits, n] of the encoder outputs."""
    _dev(x, torch.float32, "x")
    _dev(gc, torch.float32, "gc")
    if gx is None:
        gx = torch.empty(x.numel(), dtype=torch.float32, device=x.device)
    _check(lib.qnn_mbit_encoder_backward(_ptr(x), _ptr(gc), x.numel(), bits, float(r), _ptr(gx), _stream(stream)),
           "qnn_mbit_encoder_backward")
    return gx


def _workspace(nbytes: int, device, workspace):
    if workspace is None:
        workspace = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=device)
    return workspace


def bgemm_backward_data(g: torch.Tensor, w_planes: torch.Tensor, k: int, wb: int, alpha: float,
                        x: torch.Tensor | None = None, ab: int = 1, r: float = 1.0, out: torch.Tensor | None = None,
                        workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Algorithm 1 backward, activation side: g fp32 [m, n], w_planes [n, wb, row_words(k)] -> fp32 [m, k]
    (G, or the gradient through the encoder when x is given)."""
    _dev(g, torch.float32, "g")
    m, n = g.shape
    if out is None:
        out = torch.empty((m, k), dtype=torch.float32, device=g.device)
    ws = _workspace(lib.qnn_bgemm_backward_data_workspace(m, n, k), g.device, workspace)
    _check(lib.qnn_bgemm_backward_data(_ptr(g), _ptr(w_planes), m, n, k, wb, float(alpha), _ptr(x), ab, float(r),
                                       _ptr(out), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "qnn_bgemm_backward_data")
    return out


def bgemm_backward_weights(g: torch.Tensor, a_planes: torch.Tensor, k: int, ab: int, alpha: float,
                           gw: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Algorithm 1 backward, weight side: g fp32 [m, n], a_planes [m, ab, row_words(k)] -> GW fp32 [n, k]."""
    _dev(g, torch.float32, "g")
    m, n = g.shape
    if gw is None:
        gw = torch.empty((n, k), dtype=torch.float32, device=g.device)
    ws = _workspace(lib.qnn_bgemm_backward_weights_workspace(m, n, k), g.device, workspace)
    _check(lib.qnn_bgemm_backward_weights(_ptr(g), _ptr(a_planes), m, n, k, ab, float(alpha), _ptr(gw), _ptr(ws),
                                          ws.numel() * ws.element_size(), _stream(stream)), "qnn_bgemm_backward_weights")
    return gw


def bconv2d_backward_data(g: torch.Tensor, w_packed: torch.Tensor, wb: int, H: int, W: int, C: int, R: int, S: int,
                          stride: int, pad: int, alpha: float, x: torch.Tensor | None = None, ab: int = 1, r: float = 1.0,
                          out: torch.Tensor | None = None, workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Algorithm 1 backward of a convolution, activation side: g fp32 [N, Ho, Wo, Cout], packed weights -> fp32 [N, H, W, C]."""
    _dev(g, torch.float32, "g")
    N, Cout = g.shape[0], g.shape[3]
    if out is None:
        out = torch.empty((N, H, W, C), dtype=torch.float32, device=g.device)
    ws = _workspace(lib.qnn_bconv2d_backward_data_workspace(N, H, W, C, Cout, R, S, stride, pad), g.device, workspace)
    _check(lib.qnn_bconv2d_backward_data(_ptr(g), _ptr(w_packed), wb, N, H, W, C, Cout, R, S, stride, pad, float(alpha),
                                         _ptr(x), ab, float(r), _ptr(out), _ptr(ws), ws.numel() * ws.element_size(),
                                         _stream(stream)), "qnn_bconv2d_backward_data")
    return out


def bconv2d_backward_weights(g: torch.Tensor, a_planes: torch.Tensor, ab: int, H: int, W: int, C: int, R: int, S: int,
                             stride: int, pad: int, alpha: float, gw: torch.Tensor | None = None,
                             workspace: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """Algorithm 1 backward of a convolution, weight side: g fp32 [N, Ho, Wo, Cout], a_planes [N*H*W, ab, row_words(C)]
    -> GW fp32 [Cout, R, S, C]."""
    _dev(g, torch.float32, "g")
    N, Cout = g.shape[0], g.shape[3]
    if gw is None:
        gw = torch.empty((Cout, R, S, C), dtype=torch.float32, device=g.device)
    ws = _workspace(lib.qnn_bconv2d_backward_weights_workspace(N, H, W, C, Cout, R, S, stride, pad), g.device, workspace)
    _check(lib.qnn_bconv2d_backward_weights(_ptr(g), _ptr(a_planes), ab, N, H, W, C, Cout, R, S, stride, pad, float(alpha),
                                            _ptr(gw), _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)),
           "qnn_bconv2d_backward_weights")
    return gw


def unpack_codes_f32(planes: torch.Tensor, rows: int, k: int, bits: int, transpose: bool = False, stream=None) -> torch.Tensor:
    """Planes [rows, bits, row_words(k)] -> odd codes as fp32 [rows, k] (or [k, rows] when transpose)."""
    out = torch.empty((k, rows) if transpose else (rows, k), dtype=torch.float32, device=planes.device)
    _check(lib.qnn_unpack_codes_f32(_ptr(planes), rows, k, bits, int(transpose), _ptr(out), rows if transpose else k,
                                    _stream(stream)), "qnn_unpack_codes_f32")
    return out


def bgemm_int8_tensor(a_planes: torch.Tensor, ab: int, w_packed: torch.Tensor, wb: int, Mg: int, Ng: int, Kg: int,
                      alpha: float, want_acc: bool = True, out: torch.Tensor | None = None, acc: torch.Tensor | None = None,
                      workspace: torch.Tensor | None = None, stream=None):
    """Comparison path: the product of bgemm as one int8 tensor-core GEMM on the unpacked codes -> (out fp32, acc int32)."""
    dev = a_planes.device
    if out is None:
        out = torch.empty((Mg, Ng), dtype=torch.float32, device=dev)
    if acc is None and want_acc:
        acc = torch.empty((Mg, Ng), dtype=torch.int32, device=dev)
    ws = _workspace(lib.qnn_bgemm_int8_tensor_workspace(Mg, Ng, Kg), dev, workspace)
    _check(lib.qnn_bgemm_int8_tensor(_ptr(a_planes), ab, _ptr(w_packed), wb, Mg, Ng, Kg, float(alpha), _ptr(acc), _ptr(out),
                                     _ptr(ws), ws.numel() * ws.element_size(), _stream(stream)), "qnn_bgemm_int8_tensor")
    return out, acc


def tensor_path_status() -> int:
    """Synchronises; 0, or raises QnnError(QNN_E_DEVICE) when a tensor-path kernel gave up a bounded wait."""
    st = C.c_uint(0)
    _check(lib.qnn_tensor_path_status(C.byref(st)), "qnn_tensor_path_status")
    return st.value


def last_device_status() -> tuple[int, int]:
    """Synchronises; returns (return code, status word) of qnn_last_device_status without raising: (QNN_OK, 0), or
    (QNN_E_DEVICE, 1 + id of the wait that gave up).  Reading clears the record."""
    st = C.c_uint(0)
    rc = lib.qnn_last_device_status(C.byref(st))
    return rc, st.value


def selftest_bounded_wait(poll_limit: int = 1024, stream=None) -> None:
    """Enqueues the library's bounded-wait self-test (a wait that runs out on purpose and ends normally)."""
    _check(lib.qnn_selftest_bounded_wait(int(poll_limit), _stream(stream)), "qnn_selftest_bounded_wait")


def absmax_f32(x: torch.Tensor, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    _dev(x, torch.float32, "x")
    if out is None:
        out = torch.empty(1, dtype=torch.float32, device=x.device)
    _check(lib.qnn_absmax_f32(_ptr(x), x.numel(), _ptr(out), _stream(stream)), "qnn_absmax_f32")
    return out


def fc_forward_host(x_host: torch.Tensor, ab: int, scale_a: float, flags: int, w_packed: torch.Tensor, wb: int,
                    Ng: int, alpha: float, out_host: torch.Tensor, x_dev: torch.Tensor, planes_dev: torch.Tensor,
                    out_dev: torch.Tensor, stream=None) -> torch.Tensor:
    Mg, Kg = x_host.shape
    _check(lib.qnn_fc_forward_host(_ptr(x_host), Mg, Kg, ab, float(scale_a), flags, _ptr(w_packed), wb, Ng,
                                   float(alpha), _ptr(out_host), _ptr(x_dev), _ptr(planes_dev), _ptr(out_dev),
                                   _stream(stream)), "qnn_fc_forward_host")
    return out_host


def fc_forward_host_pipelined(x_host: torch.Tensor, ab: int, scale_a: float, flags: int, w_packed: torch.Tensor, wb: int,
                              Ng: int, alpha: float, out_host: torch.Tensor, x_dev: torch.Tensor,
                              planes_dev: torch.Tensor, out_dev: torch.Tensor, rows_per_chunk: int, streams,
                              join: bool = True) -> torch.Tensor:
    """Row-chunked FC layer from pinned host memory over several torch streams.  The streams are made to wait
    for the current stream first, and (join=True) the current stream waits for all of them afterwards.  With
    join=False consecutive calls on the same streams pipeline into each other (chunk i of the next call follows
    chunk i of this one on its stream); the caller joins the streams before reading out_host."""
    Mg, Kg = x_host.shape
    cur = torch.cuda.current_stream()
    for s in streams:
        s.wait_stream(cur)
    arr = (C.c_void_p * len(streams))(*[s.cuda_stream for s in streams])
    _check(lib.qnn_fc_forward_host_pipelined(_ptr(x_host), Mg, Kg, ab, float(scale_a), flags, _ptr(w_packed), wb, Ng,
                                             float(alpha), _ptr(out_host), _ptr(x_dev), _ptr(planes_dev), _ptr(out_dev),
                                             rows_per_chunk, arr, len(streams)), "qnn_fc_forward_host_pipelined")
    if join:
        for s in streams:
            cur.wait_stream(s)
    return out_host


def fc_forward_noalloc(x: torch.Tensor, ab: int, scale_a: float, flags: int, w_packed: torch.Tensor, wb: int, Ng: int,
                       alpha: float, out: torch.Tensor | None = None, stream=None) -> torch.Tensor:
    """FC layer for callers that cannot allocate: the activation planes live in the library's built-in
    buffer (at most NOALLOC_SCRATCH_BYTES of planes).  Only `out`, if not given, is allocated here, by torch."""
    _dev(x, torch.float32, "x")
    Mg, Kg = x.shape
    if out is None:
        out = torch.empty((Mg, Ng), dtype=torch.float32, device=x.device)
    _check(lib.qnn_fc_forward_noalloc(_ptr(x), Mg, Kg, x.stride(0), ab, float(scale_a), flags, _ptr(w_packed), wb, Ng,
                                      float(alpha), _ptr(out), out.stride(0), _stream(stream)),
           "qnn_fc_forward_noalloc")
    return out


def probe_bitops(variant: int, iters: int, blocks: int, sink: torch.Tensor, stream=None) -> float:
    """Enqueue the register-resident bit-op probe; returns the number of 32-bit word operations it performs."""
    ops = C.c_double(0.0)
    _check(lib.qnn_probe_bitops(variant, iters, blocks, _ptr(sink), C.byref(ops), _stream(stream)),
           "qnn_probe_bitops")
    return ops.value


def popcounts_per_output(ab: int, wb: int, conv: bool, R: int, S: int, C: int, Cout: int) -> int:
    """Popcount instructions per output element of the kernel that serves such a layer (FC: R = S = 1, C = Kg)."""
    n = lib.qnn_popcounts_per_output(ab, wb, 1 if conv else 0, R, S, C, Cout)
    if n <= 0:
        raise QnnError(E_ARG, "qnn_popcounts_per_output")
    return int(n)


def probe_copy(dst: torch.Tensor, src: torch.Tensor, stream=None) -> int:
    nbytes = src.numel() * src.element_size()
    _check(lib.qnn_probe_copy(_ptr(dst), _ptr(src), nbytes, _stream(stream)), "qnn_probe_copy")
    return nbytes


def weights_views(packed: torch.Tensor, n_out: int, taps: int, c_in: int, bits: int):
    """Split a packed-weights blob into (planes int32 [n_out, bits, row_words], tapsum int32 [n_out, taps])."""
    kw = weights_row_words(taps, c_in)
    nplane = n_out * bits * kw
    as_i32 = packed.view(torch.int32)
    return as_i32[:nplane].view(n_out, bits, kw), as_i32[nplane:nplane + n_out * taps].view(n_out, taps)


def probe_naive_sgemm(a: torch.Tensor, b: torch.Tensor, c: torch.Tensor = None, stream=None) -> torch.Tensor:
    """c = a @ b by the plain one-thread-per-output fp32 kernel (comparison line of Section 5.4); a [m, k], b [k, n]."""
    m, k = a.shape
    n = b.shape[1]
    if b.shape[0] != k or a.dtype != torch.float32 or b.dtype != torch.float32:
        raise QnnError(E_ARG, "qnn_probe_naive_sgemm")
    if not (a.is_contiguous() and b.is_contiguous()):
        raise QnnError(E_ARG, "qnn_probe_naive_sgemm: dense row-major operands")
    if c is None:
        c = torch.empty((m, n), dtype=torch.float32, device=a.device)
    if tuple(c.shape) != (m, n) or c.dtype != torch.float32 or not c.is_contiguous():
        raise QnnError(E_ARG, "qnn_probe_naive_sgemm: dense row-major [m, n] fp32 output")
    _check(lib.qnn_probe_naive_sgemm(_ptr(a), _ptr(b), _ptr(c), m, n, k, _stream(stream)), "qnn_probe_naive_sgemm")
    return c

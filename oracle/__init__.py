"""CPU oracle for the {-1,+1}-decomposed quantized layer -- TEST INFRASTRUCTURE.

This package is not part of the product.  Only the test-suite, the smoke check
and the benchmark's CPU-baseline leg may import it.  It wraps ``qnn_oracle.c``
(plain C, compiled here with gcc) behind numpy arrays; it shares no code with the
CUDA library and never calls it.

What each function follows in the paper:

* ``quantize``     -- code space of Eq. 7 / Section 3.2, interval ownership of Table 2,
                      clamp of Eq. 15.
* ``pack_planes``  -- bit-plane storage of Eq. 3 / Eq. 7, one bit per element per plane.
* ``fc`` / ``conv2d`` (and their ``_sampled`` forms) -- Op(EnC(x), EnC(w)) of Eq. 9:
                      the plain integer product that Eq. 8 reproduces exactly.
* ``scale``        -- the fixed scaling factor of Eq. 9 / Alg. 1 forward pass.
* ``mbit_encoder_forward`` / ``mbit_encoder_backward`` -- trigonometric encoder of Eq. 10 and its derivative, Eq. 12.
* ``affine``       -- per-feature affine that replaces the scale when batch normalisation follows (Section 3.2).
* ``conv_backward_data`` / ``conv_backward_weights`` -- Algorithm 1's backward products with forward() a convolution.
* ``eq16_speedup`` -- the paper's analytic speed-up model S_MK (Eq. 16, Section 4.6), plain arithmetic.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "qnn_oracle.c"
_LIB = _HERE / "libqnn_oracle.so"
_lib = None


def build(force: bool = False) -> Path:
    """Compile qnn_oracle.c into libqnn_oracle.so next to it (gcc -O2, OpenMP)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call([
            "gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
            "-Wall", "-Wextra", "-o", str(tmp), str(_SRC), "-lm",
        ])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(str(_LIB))
        c = ctypes
        p = c.c_void_p
        lib.oracle_num_threads.restype = c.c_int
        lib.oracle_row_words.restype = c.c_size_t
        lib.oracle_row_words.argtypes = [c.c_size_t]
        lib.oracle_quantize.argtypes = [p, c.c_size_t, c.c_int, c.c_float, c.c_int, p]
        lib.oracle_pack_planes.argtypes = [p, c.c_size_t, c.c_size_t, c.c_int, p]
        lib.oracle_fc.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_size_t, p]
        lib.oracle_fc_sampled.argtypes = [p, p, c.c_size_t, c.c_size_t, p, p, p]
        lib.oracle_fc_bitplanes.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_int, c.c_int, p]
        lib.oracle_conv_out_dim.argtypes = [c.c_int] * 4
        lib.oracle_conv_backward_data.argtypes = [p, p] + [c.c_int] * 11 + [c.c_float, p]
        lib.oracle_conv_backward_weights.argtypes = [p, p] + [c.c_int] * 11 + [c.c_float, p]
        lib.oracle_conv2d.argtypes = [p, p] + [c.c_int] * 9 + [p]
        lib.oracle_conv2d_sampled.argtypes = [p, p] + [c.c_int] * 9 + [c.c_size_t, p, p, p]
        lib.oracle_scale.argtypes = [p, c.c_size_t, c.c_float, p]
        lib.oracle_conv2d_general.argtypes = [p, p] + [c.c_int] * 12 + [p]
        lib.oracle_mbit_encoder_forward.argtypes = [p, c.c_size_t, c.c_int, c.c_float, p]
        lib.oracle_mbit_encoder_backward.argtypes = [p, p, c.c_size_t, c.c_int, c.c_float, p]
        lib.oracle_fc_backward_data.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_int, c.c_int, c.c_float, p]
        lib.oracle_fc_backward_weights.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_int, c.c_int, c.c_float, p]
        lib.oracle_fc_backward_data_sampled.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_int, c.c_int, c.c_float,
                                                        c.c_size_t, p, p, p]
        lib.oracle_fc_backward_weights_sampled.argtypes = [p, p, c.c_size_t, c.c_size_t, c.c_size_t, c.c_int, c.c_int,
                                                           c.c_float, c.c_size_t, p, p, p]
        lib.oracle_affine.argtypes = [p, c.c_size_t, c.c_size_t, p, p]
        _lib = lib
    return _lib


def _ptr(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _check(rc: int, what: str):
    if rc != 0:
        raise ValueError(f"oracle {what} failed with status {rc}")


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def row_words(k: int) -> int:
    return int(_load().oracle_row_words(k))


def quantize(x: np.ndarray, bits: int, scale, relu: bool = False) -> np.ndarray:
    """Real tensor -> odd integer codes (int16), same shape."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    q = np.empty(x.shape, dtype=np.int16)
    _check(_load().oracle_quantize(_ptr(x), x.size, bits, float(np.float32(scale)), int(relu), _ptr(q)),
           "quantize")
    return q


def pack_planes(q: np.ndarray, bits: int) -> np.ndarray:
    """Codes [rows, k] -> canonical planes uint32 [rows, bits, row_words(k)]."""
    q = np.ascontiguousarray(q, dtype=np.int16)
    rows, k = q.shape
    out = np.empty((rows, bits, row_words(k)), dtype=np.uint32)
    _check(_load().oracle_pack_planes(_ptr(q), rows, k, bits, _ptr(out)), "pack_planes")
    return out


def fc(qa: np.ndarray, qw: np.ndarray) -> np.ndarray:
    """qa [Mg, Kg], qw [Ng, Kg] -> int32 [Mg, Ng]."""
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    Mg, Kg = qa.shape
    Ng, Kg2 = qw.shape
    assert Kg == Kg2
    acc = np.empty((Mg, Ng), dtype=np.int32)
    _check(_load().oracle_fc(_ptr(qa), _ptr(qw), Mg, Ng, Kg, _ptr(acc)), "fc")
    return acc


def fc_bitplanes(a_planes: np.ndarray, w_planes: np.ndarray, Kg: int) -> np.ndarray:
    """Eq. 8 on packed planes: a_planes [Mg, ab, row_words(Kg)], w_planes [Ng, wb, row_words(Kg)] -> int32 [Mg, Ng]."""
    a_planes = np.ascontiguousarray(a_planes, dtype=np.uint32)
    w_planes = np.ascontiguousarray(w_planes, dtype=np.uint32)
    Mg, ab, kw = a_planes.shape
    Ng, wb, kw2 = w_planes.shape
    assert kw == kw2 == row_words(Kg)
    acc = np.empty((Mg, Ng), dtype=np.int32)
    _check(_load().oracle_fc_bitplanes(_ptr(a_planes), _ptr(w_planes), Mg, Ng, Kg, ab, wb, _ptr(acc)), "fc_bitplanes")
    return acc


def fc_sampled(qa: np.ndarray, qw: np.ndarray, rows, cols) -> np.ndarray:
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    assert rows.shape == cols.shape and qa.shape[1] == qw.shape[1]
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < qa.shape[0])
    assert cols.size == 0 or (cols.min() >= 0 and cols.max() < qw.shape[0])
    acc = np.empty(rows.shape, dtype=np.int32)
    _check(_load().oracle_fc_sampled(_ptr(qa), _ptr(qw), qa.shape[1], rows.size, _ptr(rows), _ptr(cols),
                                     _ptr(acc)), "fc_sampled")
    return acc


def conv_out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return int(_load().oracle_conv_out_dim(size, k, stride, pad))


def conv2d(qa: np.ndarray, qw: np.ndarray, stride: int, pad: int) -> np.ndarray:
    """qa [N,H,W,C], qw [Cout,R,S,C] -> int32 [N,Ho,Wo,Cout]; zero padding of the codes."""
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    N, H, W, C = qa.shape
    Cout, R, S, C2 = qw.shape
    assert C == C2
    Ho, Wo = conv_out_dim(H, R, stride, pad), conv_out_dim(W, S, stride, pad)
    acc = np.empty((N, Ho, Wo, Cout), dtype=np.int32)
    _check(_load().oracle_conv2d(_ptr(qa), _ptr(qw), N, H, W, C, Cout, R, S, stride, pad, _ptr(acc)),
           "conv2d")
    return acc


def conv2d_sampled(qa: np.ndarray, qw: np.ndarray, stride: int, pad: int, rows, cols) -> np.ndarray:
    """Outputs at (m, co) pairs, m = (n*Ho + ho)*Wo + wo."""
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    N, H, W, C = qa.shape
    Cout, R, S, C2 = qw.shape
    assert C == C2 and rows.shape == cols.shape
    Ho, Wo = conv_out_dim(H, R, stride, pad), conv_out_dim(W, S, stride, pad)
    assert rows.size == 0 or (rows.min() >= 0 and rows.max() < N * Ho * Wo)
    assert cols.size == 0 or (cols.min() >= 0 and cols.max() < Cout)
    acc = np.empty(rows.shape, dtype=np.int32)
    _check(_load().oracle_conv2d_sampled(_ptr(qa), _ptr(qw), N, H, W, C, Cout, R, S, stride, pad,
                                         rows.size, _ptr(rows), _ptr(cols), _ptr(acc)), "conv2d_sampled")
    return acc


def scale(acc: np.ndarray, alpha) -> np.ndarray:
    """float32(acc) * alpha, one rounding each."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    out = np.empty(acc.shape, dtype=np.float32)
    _check(_load().oracle_scale(_ptr(acc), acc.size, float(np.float32(alpha)), _ptr(out)), "scale")
    return out


def affine(y: np.ndarray, gamma: np.ndarray, beta: np.ndarray | None = None) -> np.ndarray:
    """y[..., n] -> fma(y, gamma[n], beta[n]) in binary32 (last axis = features); returns a new array."""
    out = np.ascontiguousarray(y, dtype=np.float32).copy()
    gamma = np.ascontiguousarray(gamma, dtype=np.float32)
    Ng = out.shape[-1]
    assert gamma.shape == (Ng,)
    if beta is not None:
        beta = np.ascontiguousarray(beta, dtype=np.float32)
        assert beta.shape == (Ng,)
    _check(_load().oracle_affine(_ptr(out), out.size // Ng, Ng, _ptr(gamma), _ptr(beta) if beta is not None else None),
           "affine")
    return out


def conv_general_out_dim(size: int, k: int, stride: int, pad: int, dil: int, transposed: bool, out_pad: int = 0) -> int:
    if not transposed:
        return (size + 2 * pad - dil * (k - 1) - 1) // stride + 1
    return (size - 1) * stride - 2 * pad + dil * (k - 1) + 1 + out_pad


def conv2d_general(qa: np.ndarray, qw: np.ndarray, stride: int, pad: int, dil: int = 1, transposed: bool = False,
                   out_pad: int = 0) -> np.ndarray:
    """Dilated or transposed convolution of codes: qa [N,H,W,C], qw [Cout,R,S,C] -> int32 [N,Ho,Wo,Cout]."""
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    N, H, W, C = qa.shape
    Cout, R, S, C2 = qw.shape
    assert C == C2
    Ho = conv_general_out_dim(H, R, stride, pad, dil, transposed, out_pad)
    Wo = conv_general_out_dim(W, S, stride, pad, dil, transposed, out_pad)
    acc = np.empty((N, Ho, Wo, Cout), dtype=np.int32)
    _check(_load().oracle_conv2d_general(_ptr(qa), _ptr(qw), N, H, W, C, Cout, R, S, stride, pad, dil, int(transposed),
                                         out_pad, _ptr(acc)), "conv2d_general")
    return acc


def mbit_encoder_forward(x: np.ndarray, bits: int, r: float = 1.0) -> np.ndarray:
    """Eq. 10: returns c float32 [bits, n] with c[m-1] = phi_M^m(x / r) in {-1, 0, +1}."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    c = np.empty((bits, x.size), dtype=np.float32)
    _check(_load().oracle_mbit_encoder_forward(_ptr(x), x.size, bits, float(np.float32(r)), _ptr(c)), "mbit_encoder_forward")
    return c


def mbit_encoder_backward(x: np.ndarray, gc: np.ndarray, bits: int, r: float = 1.0) -> np.ndarray:
    """Eq. 12: gradient with respect to x (float64 [n]) given gradients gc [bits, n] of the encoder outputs."""
    x = np.ascontiguousarray(x, dtype=np.float32).reshape(-1)
    gc = np.ascontiguousarray(gc, dtype=np.float32)
    assert gc.shape == (bits, x.size)
    gx = np.empty(x.size, dtype=np.float64)
    _check(_load().oracle_mbit_encoder_backward(_ptr(x), _ptr(gc), x.size, bits, float(np.float32(r)), _ptr(gx)),
           "mbit_encoder_backward")
    return gx


def fc_backward_data(g: np.ndarray, qw: np.ndarray, ab: int, wb: int, alpha: float) -> np.ndarray:
    """Algorithm 1, backward: g [Mg, Ng] = dC/da, qw [Ng, Kg] -> float64 [ab, Mg, Kg], entry m-1 = g_{a^m}."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    (Mg, Ng), (Ng2, Kg) = g.shape, qw.shape
    assert Ng == Ng2
    ga = np.empty((ab, Mg, Kg), dtype=np.float64)
    _check(_load().oracle_fc_backward_data(_ptr(g), _ptr(qw), Mg, Ng, Kg, ab, wb, float(np.float32(alpha)), _ptr(ga)),
           "fc_backward_data")
    return ga


def fc_backward_weights(g: np.ndarray, qa: np.ndarray, ab: int, wb: int, alpha: float) -> np.ndarray:
    """Algorithm 1, backward: g [Mg, Ng], qa [Mg, Kg] -> float64 [wb, Ng, Kg], entry j-1 = g_{W^j}."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    (Mg, Ng), (Mg2, Kg) = g.shape, qa.shape
    assert Mg == Mg2
    gw = np.empty((wb, Ng, Kg), dtype=np.float64)
    _check(_load().oracle_fc_backward_weights(_ptr(g), _ptr(qa), Mg, Ng, Kg, ab, wb, float(np.float32(alpha)), _ptr(gw)),
           "fc_backward_weights")
    return gw


def fc_backward_data_sampled(g, qw, ab: int, wb: int, alpha: float, rows, cols) -> np.ndarray:
    """g_{a^m} at (row, col) pairs: float64 [ab, count]."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    Ng, Kg = qw.shape
    assert g.shape[1] == Ng and rows.max() < g.shape[0] and cols.max() < Kg and rows.min() >= 0 and cols.min() >= 0
    out = np.empty((ab, rows.size), dtype=np.float64)
    _check(_load().oracle_fc_backward_data_sampled(_ptr(g), _ptr(qw), Ng, Kg, ab, wb, float(np.float32(alpha)), rows.size,
                                                   _ptr(rows), _ptr(cols), _ptr(out)), "fc_backward_data_sampled")
    return out


def fc_backward_weights_sampled(g, qa, ab: int, wb: int, alpha: float, rows, cols) -> np.ndarray:
    """g_{W^j} at (n, k) pairs: float64 [wb, count]."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    rows = np.ascontiguousarray(rows, dtype=np.int64)
    cols = np.ascontiguousarray(cols, dtype=np.int64)
    Mg, Kg = qa.shape
    Ng = g.shape[1]
    assert g.shape[0] == Mg and rows.max() < Ng and cols.max() < Kg and rows.min() >= 0 and cols.min() >= 0
    out = np.empty((wb, rows.size), dtype=np.float64)
    _check(_load().oracle_fc_backward_weights_sampled(_ptr(g), _ptr(qa), Mg, Ng, Kg, ab, wb, float(np.float32(alpha)),
                                                      rows.size, _ptr(rows), _ptr(cols), _ptr(out)),
           "fc_backward_weights_sampled")
    return out


def conv_backward_data(g: np.ndarray, qw: np.ndarray, hw, stride: int, pad: int, ab: int, wb: int, alpha: float) -> np.ndarray:
    """Algorithm 1, backward, convolution: g [N, Ho, Wo, Cout] = dC/d(out), qw [Cout, R, S, C], hw = (H, W) of the
    layer's input -> float64 [ab, N, H, W, C], entry m-1 = g_{a^m}."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qw = np.ascontiguousarray(qw, dtype=np.int16)
    N, Ho, Wo, Cout = g.shape
    Cout2, R, S, C = qw.shape
    H, W = hw
    assert Cout == Cout2 and Ho == conv_out_dim(H, R, stride, pad) and Wo == conv_out_dim(W, S, stride, pad)
    ga = np.empty((ab, N, H, W, C), dtype=np.float64)
    _check(_load().oracle_conv_backward_data(_ptr(g), _ptr(qw), N, H, W, C, Cout, R, S, stride, pad, ab, wb,
                                         float(np.float32(alpha)), _ptr(ga)), "conv_backward_data")
    return ga


def conv_backward_weights(g: np.ndarray, qa: np.ndarray, rs, stride: int, pad: int, ab: int, wb: int, alpha: float) -> np.ndarray:
    """Algorithm 1, backward, convolution: g [N, Ho, Wo, Cout], qa [N, H, W, C], rs = (R, S) of the kernel
    -> float64 [wb, Cout, R, S, C], entry j-1 = g_{W^j}."""
    g = np.ascontiguousarray(g, dtype=np.float32)
    qa = np.ascontiguousarray(qa, dtype=np.int16)
    N, Ho, Wo, Cout = g.shape
    N2, H, W, C = qa.shape
    R, S = rs
    assert N == N2 and Ho == conv_out_dim(H, R, stride, pad) and Wo == conv_out_dim(W, S, stride, pad)
    gw = np.empty((wb, Cout, R, S, C), dtype=np.float64)
    _check(_load().oracle_conv_backward_weights(_ptr(g), _ptr(qa), N, H, W, C, Cout, R, S, stride, pad, ab, wb,
                                            float(np.float32(alpha)), _ptr(gw)), "conv_backward_weights")
    return gw


def eq16_speedup(n: int, m_bits: int, k_bits: int, gamma: float = 1.91, beta: float | None = None, reg_len: int = 64):
    """Eq. 16 (Section 4.6): modelled speed-up S_MK of an M-bit x K-bit bit-plane dot product of length n over
    n multiply-accumulates.  The numerator is n MACs, each worth gamma bitwise operations; the denominator charges
    each of the M*K plane pairs gamma + 2*ceil(n/L) operations (xnor and bit-count per L-element register word)
    and the M*K - 1 additions that combine the pairs beta each.  The paper takes gamma = 1.91, L = 64 and
    beta = gamma/2 (the default here when beta is None)."""
    if beta is None:
        beta = gamma / 2.0
    pairs = m_bits * k_bits
    words = -(-int(n) // int(reg_len))
    return (n * gamma) / (pairs * (gamma + 2 * words) + (pairs - 1) * beta)

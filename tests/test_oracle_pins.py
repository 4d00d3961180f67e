"""Pins of the CPU oracle against what the paper and the mathematics fix.

Nothing here calls the CUDA library.  Every expected value is either printed in
the paper (Table 2, the 1/9 factor of Fig. 1), a closed form, an independent
definition (the trigonometric encoder of Eq. 10, a bit-level evaluation of Eq. 8,
exact rational arithmetic), or a library routine on a special case (numpy matmul,
torch conv2d on the integer codes in float64).
"""
from fractions import Fraction
import math

import numpy as np
import pytest

import oracle


def codes_to_t(q, bits):
    return (q.astype(np.int64) + (2 ** bits - 1)) // 2


# ----------------------------------------------------------------------------- quantizer

def _parse_frac(s):
    return Fraction(s)


def test_table2_intervals_and_states(golden_dir):
    """Table 2: interval ownership, quantized numbers and encoded states for 2 bits on [-1, 1]."""
    rows = []
    for line in (golden_dir / "table2_2bit.txt").read_text().splitlines():
        if not line.strip() or line.startswith("#"):
            continue
        lo, lo_c, hi, hi_c, num, den, sh, sl = line.split()
        rows.append((_parse_frac(lo), int(lo_c), _parse_frac(hi), int(hi_c), Fraction(int(num), int(den)),
                     int(sh), int(sl)))
    assert len(rows) == 4
    # r = 3 makes grid step s = 1 and every interval end exactly representable (x_table = x/3).
    r = 3.0
    for lo, lo_c, hi, hi_c, qv, sh, sl in rows:
        pts = [lo + (hi - lo) * Fraction(i, 16) for i in range(17)]
        for p in pts:
            if (p == lo and not lo_c) or (p == hi and not hi_c):
                continue
            x = np.array([float(p * 3)], dtype=np.float32)
            assert Fraction(float(x[0])) == p * 3 or p not in (lo, hi)
            q = int(oracle.quantize(x, 2, r / 3.0)[0])
            assert Fraction(q, 3) == qv, (p, q)
            planes = oracle.pack_planes(np.array([[q]], dtype=np.int16), 2)
            low = 1 if planes[0, 0, 0] & 1 else -1
            high = 1 if planes[0, 1, 0] & 1 else -1
            assert (high, low) == (sh, sl)
            assert low + 2 * high == q            # x = x_1 + 2 x_2 (Section 3.2)


def test_table2_exact_ties_at_r3():
    x = np.array([-3, -2.5, -2, -1, -0.5, 0, 0.5, 1, 2, 2.5, 3], dtype=np.float32)
    want = [-3, -3, -3, -1, -1, -1, 1, 1, 3, 3, 3]
    assert oracle.quantize(x, 2, 1.0).tolist() == want
    # -0.0 is zero: it belongs to "(-2/3, 0]"
    assert oracle.quantize(np.array([-0.0], dtype=np.float32), 2, 1.0).tolist() == [-1]


@pytest.mark.parametrize("bits", range(1, 9))
def test_grid_points_are_fixed_points_and_ties_go_outward(bits):
    A = 2 ** bits - 1
    s = np.float32(0.25)                       # power of two: q*s and tie points are exact
    q = np.arange(-A, A + 1, 2, dtype=np.int64)
    x = (q * float(s)).astype(np.float32)
    assert oracle.quantize(x, bits, s).tolist() == q.tolist()
    ties = np.arange(-A + 1, A, 2, dtype=np.int64)             # even integers between codes
    got = oracle.quantize((ties * float(s)).astype(np.float32), bits, s)
    want = np.where(ties > 0, ties + 1, ties - 1)               # away from zero; 0 -> -1
    assert got.tolist() == want.tolist()


@pytest.mark.parametrize("bits", range(1, 9))
def test_quantizer_nearest_monotone_symmetric_clamped(bits):
    rng = np.random.default_rng(bits)
    A = 2 ** bits - 1
    s = np.float32(0.37)
    r = float(s) * A
    x = np.sort(rng.uniform(-1.3 * r, 1.3 * r, size=20000).astype(np.float32))
    q = oracle.quantize(x, bits, s).astype(np.int64)
    assert np.all(np.abs(q) % 2 == 1) and q.min() >= -A and q.max() <= A
    assert np.all(np.diff(q) >= 0)                                   # monotone
    inside = np.abs(x.astype(np.float64)) <= r
    err = np.abs(x.astype(np.float64) - q * float(s))
    assert np.all(err[inside] <= float(s) * (1 + 1e-6))              # nearest grid point
    # strictly nearest grid point wherever the two closest grid points are not (almost) equidistant
    grid = np.arange(-A, A + 1, 2)
    d = np.abs(x.astype(np.float64)[:, None] - (grid * float(s))[None, :])
    nearest = grid[np.argmin(d, axis=1)]
    if A > 1:
        ds = np.sort(d, axis=1)
        clear = (ds[:, 1] - ds[:, 0]) > 1e-4
    else:
        clear = np.abs(x) > 1e-4
    assert np.all(q[clear] == nearest[clear])
    assert np.all(q[x > r] == A) and np.all(q[x < -r] == -A)          # end codes outside the range
    qneg = oracle.quantize(-x, bits, s).astype(np.int64)
    assert np.all(qneg[x != 0] == -q[x != 0])                         # odd symmetry away from 0


def test_relu_flag_and_nonfinite():
    x = np.array([-5.0, -0.1, 0.0, 0.1, 0.9, np.inf, -np.inf, np.nan], dtype=np.float32)
    assert oracle.quantize(x, 2, 1.0 / 3, relu=True).tolist() == [-1, -1, -1, 1, 3, 3, -1, -1]
    assert oracle.quantize(x, 2, 1.0 / 3, relu=False).tolist() == [-3, -1, -1, 1, 3, 3, -3, -3]


# ----------------------------------------------------------------------------- planes

@pytest.mark.parametrize("bits", range(1, 9))
def test_planes_match_trigonometric_encoder(bits):
    """Eq. 10: the m-th encoder output is sign(+-sin((2^M-1)/2^m * pi * x)) for x in [-1, 1]."""
    M = bits
    A = 2 ** M - 1
    rng = np.random.default_rng(100 + bits)
    x = rng.uniform(-1, 1, size=6000)
    # keep away from interval boundaries (even multiples of 1/A) where sign(sin) is 0
    dist = np.abs(x * A / 2 - np.round(x * A / 2))
    x = x[dist > 1e-3]
    xf = x.astype(np.float32)
    q = oracle.quantize(xf, M, np.float32(1.0) / np.float32(A))
    planes = oracle.pack_planes(q.reshape(1, -1), M)
    for m in range(1, M + 1):
        arg = (2 ** M - 1) / 2 ** m * math.pi * xf.astype(np.float64)
        phi = np.sign(np.sin(arg)) if m == M else np.sign(-np.sin(arg))
        words = planes[0, m - 1]
        bits_m = (words[np.arange(x.size) // 32] >> (np.arange(x.size) % 32).astype(np.uint32)) & 1
        assert np.array_equal(np.where(bits_m == 1, 1.0, -1.0), phi), (M, m)


@pytest.mark.parametrize("bits", range(1, 9))
def test_eq7_reconstruction_from_planes(bits):
    rng = np.random.default_rng(7 + bits)
    A = 2 ** bits - 1
    q = (2 * rng.integers(0, A + 1, size=(5, 77)) - A).astype(np.int16)
    planes = oracle.pack_planes(q, bits)
    k = np.arange(77)
    rec = np.zeros((5, 77), dtype=np.int64)
    for i in range(bits):
        c = ((planes[:, i, :][:, k // 32] >> (k % 32).astype(np.uint32)) & 1).astype(np.int64) * 2 - 1
        rec += (2 ** i) * c
    assert np.array_equal(rec, q)


def test_plane_layout_word_and_bit_position():
    """Element k sits in bit k%32 of word k//32; pad bits are zero; rows padded to 4 words."""
    k = 70
    q = -np.ones((2, k), dtype=np.int16) * 3        # t = 0 everywhere (2 bits)
    q[1, 37] = 3                                    # t = 3: both planes set
    q[0, 69] = 1                                    # t = 2: only plane 1
    planes = oracle.pack_planes(q, 2)
    assert planes.shape == (2, 2, 4) and oracle.row_words(k) == 4
    want = np.zeros((2, 2, 4), dtype=np.uint32)
    want[1, 0, 1] = 1 << 5
    want[1, 1, 1] = 1 << 5
    want[0, 1, 2] = 1 << 5
    assert np.array_equal(planes, want)
    ones = oracle.pack_planes(np.ones((1, k), dtype=np.int16) * 3, 2)
    assert ones[0, 0].tolist() == [0xFFFFFFFF, 0xFFFFFFFF, 0x3F, 0]
    assert oracle.row_words(128) == 4 and oracle.row_words(129) == 8 and oracle.row_words(1) == 4


@pytest.mark.parametrize("bits,ratio", [(1, 32), (2, 16), (3, 10.7), (4, 8), (5, 6.4), (6, 5.3), (7, 4.6), (8, 4)])
def test_packed_size_matches_compression_column(bits, ratio):
    """Table 3's compression column: 32/bits relative to fp32 storage."""
    rows, k = 16, 1024
    planes = oracle.pack_planes(np.ones((rows, k), dtype=np.int16), bits)
    assert abs(rows * k * 4 / planes.nbytes - ratio) < 0.05


# ----------------------------------------------------------------------------- contraction

def branch_sum_bruteforce(pa, pw, N, ab, wb):
    """Eq. 8 evaluated literally on bit planes: sum_ij 2^(i+j) * (N - 2*popcount(a_i xor w_j))."""
    Mg, Ng = pa.shape[0], pw.shape[0]
    out = np.zeros((Mg, Ng), dtype=np.int64)
    for m in range(Mg):
        for n in range(Ng):
            s = 0
            for i in range(ab):
                for j in range(wb):
                    x = np.bitwise_xor(pa[m, i], pw[n, j])
                    pc = sum(bin(int(v)).count("1") for v in x)
                    s += (1 << (i + j)) * (N - 2 * pc)
            out[m, n] = s
    return out


@pytest.mark.parametrize("ab,wb,Kg", [(1, 1, 40), (2, 2, 65), (3, 2, 33), (4, 4, 130), (2, 4, 7), (8, 8, 50), (5, 1, 96)])
def test_eq8_branch_identity(ab, wb, Kg):
    rng = np.random.default_rng(ab * 100 + wb * 10 + Kg)
    A, B = 2 ** ab - 1, 2 ** wb - 1
    qa = (2 * rng.integers(0, A + 1, size=(5, Kg)) - A).astype(np.int16)
    qw = (2 * rng.integers(0, B + 1, size=(6, Kg)) - B).astype(np.int16)
    acc = oracle.fc(qa, qw)
    assert np.array_equal(acc, branch_sum_bruteforce(oracle.pack_planes(qa, ab), oracle.pack_planes(qw, wb), Kg, ab, wb))
    # Eq. 6 / Eq. 18 form on the {0,1}-coded integers t
    ta, tw = codes_to_t(qa, ab), codes_to_t(qw, wb)
    alt = 4 * ta @ tw.T - 2 * B * ta.sum(1)[:, None] - 2 * A * tw.sum(1)[None, :] + Kg * A * B
    assert np.array_equal(acc, alt)


@pytest.mark.parametrize("ab,wb,Kg", [(1, 1, 40), (2, 2, 65), (3, 2, 33), (4, 4, 130), (2, 4, 7), (8, 8, 50), (5, 1, 96), (2, 2, 1)])
def test_fc_bitplanes_is_eq8_and_agrees_with_the_plain_definition(ab, wb, Kg):
    """The popcount form of the oracle against three things that are not itself: the literal Python evaluation of
    Eq. 8, a numpy float64 product of the codes, and the closed form for equal / opposite extreme operands."""
    rng = np.random.default_rng(ab * 1000 + wb * 37 + Kg)
    A, B = 2 ** ab - 1, 2 ** wb - 1
    qa = (2 * rng.integers(0, A + 1, size=(7, Kg)) - A).astype(np.int16)
    qw = (2 * rng.integers(0, B + 1, size=(5, Kg)) - B).astype(np.int16)
    pa, pw = oracle.pack_planes(qa, ab), oracle.pack_planes(qw, wb)
    got = oracle.fc_bitplanes(pa, pw, Kg)
    assert np.array_equal(got, branch_sum_bruteforce(pa, pw, Kg, ab, wb))
    assert np.array_equal(got.astype(np.float64), qa.astype(np.float64) @ qw.astype(np.float64).T)
    hi_a, hi_w = np.full((2, Kg), A, dtype=np.int16), np.full((3, Kg), B, dtype=np.int16)
    assert np.all(oracle.fc_bitplanes(oracle.pack_planes(hi_a, ab), oracle.pack_planes(hi_w, wb), Kg) == Kg * A * B)
    assert np.all(oracle.fc_bitplanes(oracle.pack_planes(hi_a, ab), oracle.pack_planes(-hi_w, wb), Kg) == -Kg * A * B)


def test_fc_matches_numpy_matmul_ragged():
    rng = np.random.default_rng(5)
    qa = (2 * rng.integers(0, 16, size=(37, 301)) - 15).astype(np.int16)
    qw = (2 * rng.integers(0, 8, size=(29, 301)) - 7).astype(np.int16)
    want = qa.astype(np.float64) @ qw.astype(np.float64).T
    got = oracle.fc(qa, qw)
    assert np.array_equal(got.astype(np.float64), want)
    rows = rng.integers(0, 37, size=50)
    cols = rng.integers(0, 29, size=50)
    assert np.array_equal(oracle.fc_sampled(qa, qw, rows, cols), got[rows, cols])


def test_closed_forms():
    N = 123
    for ab, wb in [(1, 1), (2, 3), (4, 4), (8, 8)]:
        A, B = 2 ** ab - 1, 2 ** wb - 1
        assert oracle.fc(np.full((2, N), A, np.int16), np.full((3, N), B, np.int16)).tolist() == [[N * A * B] * 3] * 2
        assert oracle.fc(np.full((2, N), -A, np.int16), np.full((3, N), B, np.int16)).tolist() == [[-N * A * B] * 3] * 2
    rng = np.random.default_rng(1)
    q = (2 * rng.integers(0, 8, size=(1, N)) - 7).astype(np.int16)
    assert oracle.fc(q, -q)[0, 0] == -int((q.astype(np.int64) ** 2).sum())


def test_one_bit_is_sign_xnor_popcount():
    """1-bit x 1-bit reduces to the binarized-network product: sign vectors, 2*popc(xnor) - N."""
    rng = np.random.default_rng(3)
    x = rng.standard_normal((4, 100)).astype(np.float32)
    w = rng.standard_normal((3, 100)).astype(np.float32)
    x[x == 0] = 1
    qa, qw = oracle.quantize(x, 1, 1.0), oracle.quantize(w, 1, 1.0)
    assert np.array_equal(qa, np.sign(x).astype(np.int16))
    sa, sw = x > 0, w > 0
    want = np.array([[2 * int(np.sum(~(sa[m] ^ sw[n]))) - 100 for n in range(3)] for m in range(4)])
    assert np.array_equal(oracle.fc(qa, qw), want)


def test_overflow_is_reported():
    Kg = 40000                                    # 40000 * 255 * 255 > 2^31
    qa = np.full((1, Kg), 255, np.int16)
    with pytest.raises(ValueError):
        oracle.fc(qa, qa)


# ----------------------------------------------------------------------------- scale

def test_fig1_two_bit_fc_scale_one_ninth():
    """2-bit FC on [-1,1] data: real product of the quantized numbers = integer product / 9 (Fig. 1, Eq. 19)."""
    vals = [Fraction(-1), Fraction(-1, 3), Fraction(1, 3), Fraction(1)]
    rng = np.random.default_rng(11)
    xi = rng.integers(0, 4, size=(3, 24))
    wi = rng.integers(0, 4, size=(5, 24))
    # feed points strictly inside each Table-2 interval
    centers = np.array([-0.9, -0.3, 0.3, 0.9], dtype=np.float32)
    s = np.float32(1.0) / np.float32(3.0)
    qa, qw = oracle.quantize(centers[xi], 2, s), oracle.quantize(centers[wi], 2, s)
    acc = oracle.fc(qa, qw)
    for m in range(3):
        for n in range(5):
            exact = sum(vals[xi[m, k]] * vals[wi[n, k]] for k in range(24))
            assert Fraction(int(acc[m, n]), 9) == exact
    out = oracle.scale(acc, np.float32(1.0) / np.float32(9.0))
    assert np.allclose(out, acc / 9.0, rtol=2e-7)


def test_scale_against_float_bruteforce_of_decoded_values():
    rng = np.random.default_rng(17)
    a = np.maximum(rng.standard_normal((6, 90)), 0).astype(np.float32)
    w = (0.05 * rng.standard_normal((7, 90))).astype(np.float32)
    for ab, wb in [(2, 2), (3, 4), (1, 8)]:
        sa = np.float32(np.abs(a).max()) / np.float32(2 ** ab - 1)
        sw = np.float32(np.abs(w).max()) / np.float32(2 ** wb - 1)
        qa, qw = oracle.quantize(a, ab, sa), oracle.quantize(w, wb, sw)
        alpha = np.float32(sa * sw)
        out = oracle.scale(oracle.fc(qa, qw), alpha)
        brute = (qa.astype(np.float64) * float(sa)) @ (qw.astype(np.float64) * float(sw)).T
        assert np.allclose(out, brute, rtol=1e-6, atol=1e-9)
        # the quantized layer approximates the real one (coarse sanity of grid + scale)
        assert np.abs(out - a.astype(np.float64) @ w.astype(np.float64).T).max() <= 90 * float(sa) * float(sw) * (2 ** ab) * (2 ** wb)


def test_scale_is_single_rounding():
    acc = np.array([0, 1, -1, 16777217, -2147483648, 2147483647, 123456789], dtype=np.int32)
    alpha = np.float32(0.013671875)
    want = (acc.astype(np.float32) * alpha).astype(np.float32)
    assert np.array_equal(oracle.scale(acc, alpha), want)


# ----------------------------------------------------------------------------- convolution

def im2col_zero(qa, R, S, stride, pad):
    N, H, W, C = qa.shape
    Ho, Wo = (H + 2 * pad - R) // stride + 1, (W + 2 * pad - S) // stride + 1
    padded = np.zeros((N, H + 2 * pad, W + 2 * pad, C), dtype=qa.dtype)
    padded[:, pad:pad + H, pad:pad + W] = qa
    cols = np.empty((N, Ho, Wo, R, S, C), dtype=qa.dtype)
    for r in range(R):
        for s in range(S):
            cols[:, :, :, r, s, :] = padded[:, r:r + stride * Ho:stride, s:s + stride * Wo:stride, :]
    return cols.reshape(N * Ho * Wo, R * S * C), Ho, Wo


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad", [
    (2, 5, 6, 7, 4, 3, 3, 1, 1), (1, 7, 7, 3, 5, 3, 3, 2, 1), (2, 6, 6, 9, 3, 1, 1, 2, 0),
    (1, 4, 5, 33, 2, 3, 3, 1, 0), (1, 9, 8, 4, 3, 5, 3, 2, 2), (2, 3, 3, 8, 8, 3, 3, 1, 1)])
def test_conv_equals_fc_on_explicit_im2col_and_torch(N, H, W, C, Cout, R, S, stride, pad):
    import torch
    rng = np.random.default_rng(N * 1000 + H * 100 + C)
    qa = (2 * rng.integers(0, 8, size=(N, H, W, C)) - 7).astype(np.int16)
    qw = (2 * rng.integers(0, 4, size=(Cout, R, S, C)) - 3).astype(np.int16)
    acc = oracle.conv2d(qa, qw, stride, pad)
    cols, Ho, Wo = im2col_zero(qa, R, S, stride, pad)
    assert acc.shape == (N, Ho, Wo, Cout)
    assert np.array_equal(acc.reshape(-1, Cout), oracle.fc(cols, qw.reshape(Cout, -1)))
    ref = torch.nn.functional.conv2d(torch.from_numpy(qa.astype(np.float64)).permute(0, 3, 1, 2),
                                     torch.from_numpy(qw.astype(np.float64)).permute(0, 3, 1, 2),
                                     stride=stride, padding=pad).permute(0, 2, 3, 1).numpy()
    assert np.array_equal(acc.astype(np.float64), ref)
    rows = rng.integers(0, N * Ho * Wo, size=40)
    cc = rng.integers(0, Cout, size=40)
    assert np.array_equal(oracle.conv2d_sampled(qa, qw, stride, pad, rows, cc), acc.reshape(-1, Cout)[rows, cc])


def test_conv_1x1_is_gemm_and_border_counts_valid_taps():
    rng = np.random.default_rng(2)
    qa = (2 * rng.integers(0, 4, size=(2, 4, 4, 16)) - 3).astype(np.int16)
    qw = (2 * rng.integers(0, 4, size=(6, 1, 1, 16)) - 3).astype(np.int16)
    assert np.array_equal(oracle.conv2d(qa, qw, 1, 0).reshape(-1, 6), oracle.fc(qa.reshape(-1, 16), qw.reshape(6, 16)))
    # all codes +1 (1 bit): each output counts C * (#taps inside the image); corners see 4 of 9 taps
    ones = np.ones((1, 5, 5, 8), np.int16)
    acc = oracle.conv2d(ones, np.ones((1, 3, 3, 8), np.int16), 1, 1)[0, :, :, 0]
    assert acc[0, 0] == 8 * 4 and acc[0, 2] == 8 * 6 and acc[2, 2] == 8 * 9 and acc[4, 4] == 8 * 4


# ----------------------------------------------------------------------------- per-feature affine

def test_affine_exact_cases_and_single_rounding():
    """Where the fused multiply-add is exact (small integers, power-of-two gains) the result is the integer
    arithmetic; in general it is the correctly rounded value of y*gamma + beta, i.e. within half an ulp of the
    float64 value and different from the twice-rounded product-then-sum where those differ."""
    y = np.arange(-12, 12, dtype=np.float32).reshape(4, 6)
    g = np.array([1, 2, 0.5, -4, 8, 0.25], dtype=np.float32)
    b = np.array([0, 1, -3, 5, 0.5, -0.25], dtype=np.float32)
    assert np.array_equal(oracle.affine(y, g, b), (y.astype(np.float64) * g + b).astype(np.float32))
    assert np.array_equal(oracle.affine(y, g), (y.astype(np.float64) * g).astype(np.float32))
    rng = np.random.default_rng(9)
    y = rng.standard_normal((50, 33)).astype(np.float32) * 100
    g = rng.standard_normal(33).astype(np.float32)
    b = rng.standard_normal(33).astype(np.float32)
    got = oracle.affine(y, g, b)
    exact = y.astype(np.float64) * g.astype(np.float64) + b.astype(np.float64)
    assert np.array_equal(got, exact.astype(np.float32))            # float64 holds the exact product: one rounding
    twice = (y * g).astype(np.float32) + b
    assert np.any(got != twice.astype(np.float32))                   # a plain multiply then add would differ somewhere
    assert got.shape == y.shape and np.array_equal(y, y.copy())


# ----------------------------------------------------------------------------- dilated / transposed convolution

@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad,dil,transposed,out_pad", [
    (2, 9, 8, 5, 3, 3, 3, 1, 2, 2, False, 0), (1, 11, 11, 4, 6, 3, 3, 2, 1, 3, False, 0), (1, 7, 7, 3, 2, 3, 3, 1, 1, 1, False, 0),
    (2, 5, 6, 4, 3, 3, 3, 2, 1, 1, True, 1), (1, 4, 4, 7, 5, 4, 4, 2, 1, 1, True, 0), (1, 6, 5, 3, 4, 3, 2, 3, 0, 1, True, 2),
    (1, 5, 5, 2, 3, 3, 3, 2, 2, 2, True, 0), (2, 3, 3, 6, 2, 1, 1, 2, 0, 1, True, 1)])
def test_general_conv_matches_torch(N, H, W, C, Cout, R, S, stride, pad, dil, transposed, out_pad):
    import torch
    rng = np.random.default_rng(H * 31 + C + stride)
    qa = (2 * rng.integers(0, 8, size=(N, H, W, C)) - 7).astype(np.int16)
    qw = (2 * rng.integers(0, 4, size=(Cout, R, S, C)) - 3).astype(np.int16)
    acc = oracle.conv2d_general(qa, qw, stride, pad, dil, transposed, out_pad)
    x = torch.from_numpy(qa.astype(np.float64)).permute(0, 3, 1, 2)
    if not transposed:
        wt = torch.from_numpy(qw.astype(np.float64)).permute(0, 3, 1, 2)                 # [Cout, C, R, S]
        ref = torch.nn.functional.conv2d(x, wt, stride=stride, padding=pad, dilation=dil)
        if dil == 1:
            assert np.array_equal(acc, oracle.conv2d(qa, qw, stride, pad))
    else:
        wt = torch.from_numpy(qw.astype(np.float64)).permute(3, 0, 1, 2)                 # [C, Cout, R, S]
        ref = torch.nn.functional.conv_transpose2d(x, wt, stride=stride, padding=pad, output_padding=out_pad, dilation=dil)
    assert np.array_equal(acc.astype(np.float64), ref.permute(0, 2, 3, 1).numpy())


# ----------------------------------------------------------------------------- trigonometric encoder (training side)

@pytest.mark.parametrize("bits", range(1, 9))
def test_mbit_encoder_forward_is_sign_of_sine_and_matches_the_lookup_encoder(bits):
    """Away from the zero crossings the parity rule equals sign(+-sin(k pi x)) evaluated in float64 (Eq. 10), and its
    bits are the planes of the table quantizer (Table 2 / Eq. 7) for data in [-1, 1]; at crossings it is 0."""
    rng = np.random.default_rng(50 + bits)
    A = 2 ** bits - 1
    x = rng.uniform(-1, 1, size=5000)
    x = x[np.abs(x * A / 2 - np.round(x * A / 2)) > 1e-3].astype(np.float32)
    c = oracle.mbit_encoder_forward(x, bits)
    q = oracle.quantize(x, bits, np.float32(1.0) / np.float32(A)).astype(np.int64)
    t = (q + A) // 2
    for m in range(1, bits + 1):
        arg = A / 2 ** m * math.pi * x.astype(np.float64)
        want = np.sign(np.sin(arg)) if m == bits else np.sign(-np.sin(arg))
        assert np.array_equal(c[m - 1], want.astype(np.float32)), (bits, m)
        assert np.array_equal(c[m - 1], np.where((t >> (m - 1)) & 1, 1.0, -1.0).astype(np.float32))
    # exact zero crossings give 0: x = 0 for every bit, and x = +-2, 4 for the lowest bit (k_1 * x = A * x / 2 is an integer)
    cz = oracle.mbit_encoder_forward(np.array([0.0, 2.0, -2.0, 4.0], dtype=np.float32), bits)
    assert np.all(cz[:, 0] == 0.0) and np.all(cz[0] == 0.0)


@pytest.mark.parametrize("bits", range(1, 9))
def test_mbit_encoder_forward_near_crossings_against_exact_rational_arithmetic(bits):
    """Inside the band around the zero crossings, where a float64 sine cannot be trusted to decide the sign.
    (a) Inputs x = n / 2^16: k_m * x = A * n / 2^(m+16) has at most 24 significant bits, so the binary32 product
        of Eq. 10's argument is exact and sign(sin(pi * k_m * x)) is decided by integer arithmetic alone: 0 when
        2^(m+16) divides A * n, else + on (2j, 2j+1) and - on (2j+1, 2j+2).  Every n in [-2^16, 2^16] is checked,
        which includes each crossing that is a multiple of 2^-16 and its two neighbours on that grid.
    (b) Arbitrary binary32 inputs within 1e-3 of a crossing (the band the float64 pin leaves out), including the
        floats adjacent to each crossing: the argument is y = fl32(k_m * fl32(x / r)) (the reading of Eq. 10's
        precision); numpy's IEEE binary32 operations give y, fractions.Fraction decides integer / parity exactly."""
    from fractions import Fraction
    A = 2 ** bits - 1
    n = np.arange(-2 ** 16, 2 ** 16 + 1, dtype=np.int64)
    x = (n.astype(np.float64) / 2.0 ** 16).astype(np.float32)
    assert np.array_equal(x.astype(np.float64) * 2.0 ** 16, n.astype(np.float64))
    c = oracle.mbit_encoder_forward(x, bits)
    for m in range(1, bits + 1):
        num, sh = A * n, m + 16                            # k_m * x = num / 2^sh exactly
        integer = (num & ((1 << sh) - 1)) == 0
        odd_floor = ((num >> sh) & 1) == 1                 # arithmetic shift = floor, also for negatives
        want = np.where(integer, 0.0, np.where(odd_floor, -1.0, 1.0))
        if m != bits:
            want = -want
        assert np.array_equal(c[m - 1], want.astype(np.float32)), (bits, m)
        # the same through fractions.Fraction, literally, on a handful of points around crossings
        for idx in (0, 1, 2 ** 16 - 1, 2 ** 16, 2 ** 16 + 1, 2 ** 17 - 1, 2 ** 17, 12345, 77777):
            y = Fraction(A, 2 ** m) * Fraction(float(x[idx]))
            fl = y.numerator // y.denominator
            sg = 0.0 if y.denominator == 1 else (1.0 if fl % 2 == 0 else -1.0)
            assert c[m - 1][idx] == (sg if m == bits else -sg)
    # (b) floats in the band around crossings, several ranges r
    rng = np.random.default_rng(500 + bits)
    for r in (1.0, 3.0, 0.37):
        r32 = np.float32(r)
        cross = rng.integers(-A, A + 1, size=400).astype(np.float64) * 2.0 / A * r     # crossings of the lowest plane
        xb = (cross + rng.uniform(-1e-3, 1e-3, size=cross.size) * 2.0 / A * r).astype(np.float32)
        xc = cross.astype(np.float32)
        xs = np.concatenate([xb, xc, np.nextafter(xc, np.float32(np.inf)), np.nextafter(xc, np.float32(-np.inf))])
        cb = oracle.mbit_encoder_forward(xs, bits, r)
        xn = xs / r32                                       # binary32 division
        for m in range(1, bits + 1):
            k32 = np.float32(A) / np.float32(2 ** m)       # exact
            y32 = k32 * xn                                  # binary32 product (numpy: IEEE, not the oracle's C code)
            for e in range(0, xs.size, 7):
                y = Fraction(float(y32[e]))
                fl = y.numerator // y.denominator
                sg = 0.0 if y.denominator == 1 else (1.0 if fl % 2 == 0 else -1.0)
                assert cb[m - 1][e] == (sg if m == bits else -sg), (bits, m, r, float(xs[e]))


@pytest.mark.parametrize("bits", [1, 2, 3, 5, 8])
def test_mbit_encoder_backward_is_the_derivative_of_the_sine_and_zero_outside(bits):
    """Eq. 12 is the derivative of the sine inside the sign (a straight-through estimate): compare with a central
    difference of +-sin(k pi x) in float64, and check the cut-off outside [-1, 1] and the 1/r chain factor."""
    rng = np.random.default_rng(60 + bits)
    A = 2 ** bits - 1
    x = rng.uniform(-0.99, 0.99, size=400).astype(np.float32)
    for m in range(1, bits + 1):
        gc = np.zeros((bits, x.size), dtype=np.float32)
        gc[m - 1] = 1.0
        got = oracle.mbit_encoder_backward(x, gc, bits)
        k = A / 2 ** m
        f = (lambda z: np.sin(k * math.pi * z)) if m == bits else (lambda z: -np.sin(k * math.pi * z))
        h = 1e-6
        num = (f(x.astype(np.float64) + h) - f(x.astype(np.float64) - h)) / (2 * h)
        assert np.allclose(got, num, rtol=1e-5, atol=1e-4 * k)
    xo = np.array([-1.5, 1.0000001, 2.0, -1.0, 1.0, 0.0], dtype=np.float32)
    g = oracle.mbit_encoder_backward(xo, np.ones((bits, xo.size), np.float32), bits)
    assert np.all(g[:3] == 0.0) and g[5] != 0.0
    # chain rule through the range: encoder(x / r)
    r = 3.0
    xr = (x * r).astype(np.float32)
    g1 = oracle.mbit_encoder_backward(xr, np.ones((bits, x.size), np.float32), bits, r)
    g0 = oracle.mbit_encoder_backward((xr / np.float32(r)).astype(np.float32), np.ones((bits, x.size), np.float32), bits)
    assert np.allclose(g1, g0 / r, rtol=1e-12)


# ----------------------------------------------------------------------------- backward products (Algorithm 1)

def _planes_pm1(q, bits):
    """Codes -> float64 [bits, ...] of {-1,+1} planes (plane i-1 = a^i), by Eq. 8's bit decomposition."""
    t = codes_to_t(q, bits)
    return np.stack([np.where((t >> i) & 1, 1.0, -1.0) for i in range(bits)])


def _backward_case(seed, Mg, Ng, Kg, ab, wb):
    rng = np.random.default_rng(seed)
    qa = (2 * rng.integers(0, 2 ** ab, size=(Mg, Kg)) - (2 ** ab - 1)).astype(np.int16)
    qw = (2 * rng.integers(0, 2 ** wb, size=(Ng, Kg)) - (2 ** wb - 1)).astype(np.int16)
    g = rng.standard_normal((Mg, Ng)).astype(np.float32)
    alpha = float(np.float32(0.37 / ((2 ** ab - 1) * (2 ** wb - 1))))
    return qa, qw, g, alpha


@pytest.mark.parametrize("ab,wb", [(1, 1), (2, 2), (3, 1), (2, 4), (8, 8)])
def test_backward_products_are_the_exact_change_of_the_forward_under_a_plane_flip(ab, wb):
    """The forward (the pinned integer product) is linear in every plane entry, so flipping one entry of a^m or W^j
    from -1 to +1 changes C = <g, alpha * a_hat> by exactly twice the oracle's gradient at that entry."""
    Mg, Ng, Kg = 5, 7, 9
    qa, qw, g, alpha = _backward_case(100 * ab + wb, Mg, Ng, Kg, ab, wb)
    ga = oracle.fc_backward_data(g, qw, ab, wb, alpha)
    gw = oracle.fc_backward_weights(g, qa, ab, wb, alpha)
    assert ga.shape == (ab, Mg, Kg) and gw.shape == (wb, Ng, Kg)

    def cost(qa_, qw_):
        return float(np.sum(g.astype(np.float64) * alpha * oracle.fc(qa_, qw_).astype(np.float64)))

    rng = np.random.default_rng(7)
    pa, pw = _planes_pm1(qa, ab), _planes_pm1(qw, wb)
    base = cost(qa, qw)
    for _ in range(40):
        m, r, k = rng.integers(0, ab), rng.integers(0, Mg), rng.integers(0, Kg)
        q2 = qa.copy()
        q2[r, k] -= np.int16(pa[m, r, k] * 2 * 2 ** m)              # flips plane m of that entry
        assert cost(q2, qw) - base == pytest.approx(-2 * pa[m, r, k] * ga[m, r, k], rel=1e-9, abs=1e-12)
        j, n, k = rng.integers(0, wb), rng.integers(0, Ng), rng.integers(0, Kg)
        w2 = qw.copy()
        w2[n, k] -= np.int16(pw[j, n, k] * 2 * 2 ** j)
        assert cost(qa, w2) - base == pytest.approx(-2 * pw[j, n, k] * gw[j, n, k], rel=1e-9, abs=1e-12)


@pytest.mark.parametrize("ab,wb", [(2, 2), (4, 3)])
def test_backward_products_special_cases(ab, wb):
    """A one-hot g picks out one weight row / one activation row scaled by alpha * 2^(m-1); a library matmul on the
    codes gives the same numbers; the sampled variants agree with the full ones."""
    Mg, Ng, Kg = 6, 10, 13
    qa, qw, g, alpha = _backward_case(5, Mg, Ng, Kg, ab, wb)
    e = np.zeros((Mg, Ng), dtype=np.float32)
    e[2, 3] = 1.0
    ga = oracle.fc_backward_data(e, qw, ab, wb, alpha)
    gw = oracle.fc_backward_weights(e, qa, ab, wb, alpha)
    for m in range(ab):
        want = np.zeros((Mg, Kg))
        want[2] = alpha * 2.0 ** m * qw[3]
        assert np.allclose(ga[m], want, rtol=1e-14, atol=0)
    for j in range(wb):
        want = np.zeros((Ng, Kg))
        want[3] = alpha * 2.0 ** j * qa[2]
        assert np.allclose(gw[j], want, rtol=1e-14, atol=0)
    ga = oracle.fc_backward_data(g, qw, ab, wb, alpha)
    gw = oracle.fc_backward_weights(g, qa, ab, wb, alpha)
    G = alpha * g.astype(np.float64)
    for m in range(ab):
        assert np.allclose(ga[m], 2.0 ** m * (G @ qw.astype(np.float64)), rtol=1e-12, atol=1e-15)
    for j in range(wb):
        assert np.allclose(gw[j], 2.0 ** j * (G.T @ qa.astype(np.float64)), rtol=1e-12, atol=1e-15)
    rows = np.array([0, 5, 2, 2]); cols = np.array([12, 0, 7, 8])
    assert np.array_equal(oracle.fc_backward_data_sampled(g, qw, ab, wb, alpha, rows, cols), ga[:, rows, cols])
    rows = np.array([9, 0, 4, 4])
    assert np.array_equal(oracle.fc_backward_weights_sampled(g, qa, ab, wb, alpha, rows, cols), gw[:, rows, cols])



# ---- Algorithm 1 backward with forward() a convolution --------------------------------------------------------------

def _conv_backward_case(seed, N, H, W, C, Cout, R, S, stride, pad, ab, wb):
    rng = np.random.default_rng(seed)
    qa = (2 * rng.integers(0, 2 ** ab, size=(N, H, W, C)) - (2 ** ab - 1)).astype(np.int16)
    qw = (2 * rng.integers(0, 2 ** wb, size=(Cout, R, S, C)) - (2 ** wb - 1)).astype(np.int16)
    Ho, Wo = oracle.conv_out_dim(H, R, stride, pad), oracle.conv_out_dim(W, S, stride, pad)
    g = rng.standard_normal((N, Ho, Wo, Cout)).astype(np.float32)
    alpha = float(np.float32(0.21 / ((2 ** ab - 1) * (2 ** wb - 1))))
    return qa, qw, g, alpha


@pytest.mark.parametrize("ab,wb,stride,pad", [(1, 1, 1, 1), (2, 3, 2, 1), (4, 2, 1, 0), (3, 3, 2, 2)])
def test_conv_backward_is_the_exact_change_of_the_forward_under_a_plane_flip(ab, wb, stride, pad):
    """The pinned forward convolution is linear in every plane entry: flipping one entry of a^m or W^j changes
    C = <g, alpha * conv(qa, qw)> by exactly twice the gradient there (border elements, read by fewer taps, included)."""
    N, H, W, C, Cout, R, S = 2, 6, 5, 3, 4, 3, 3
    qa, qw, g, alpha = _conv_backward_case(10 * ab + wb, N, H, W, C, Cout, R, S, stride, pad, ab, wb)
    ga = oracle.conv_backward_data(g, qw, (H, W), stride, pad, ab, wb, alpha)
    gw = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, wb, alpha)
    assert ga.shape == (ab, N, H, W, C) and gw.shape == (wb, Cout, R, S, C)

    def cost(qa_, qw_):
        return float(np.sum(g.astype(np.float64) * alpha * oracle.conv2d(qa_, qw_, stride, pad).astype(np.float64)))

    pa, pw = _planes_pm1(qa.reshape(-1, C), ab).reshape((ab,) + qa.shape), _planes_pm1(qw.reshape(-1, C), wb).reshape((wb,) + qw.shape)
    base = cost(qa, qw)
    rng = np.random.default_rng(3)
    corners = [(0, 0, 0, 0), (N - 1, H - 1, W - 1, C - 1), (0, H - 1, 0, 1)]
    for it in range(30):
        idx = corners[it] if it < len(corners) else tuple(int(rng.integers(0, d)) for d in qa.shape)
        m = int(rng.integers(0, ab))
        q2 = qa.copy()
        q2[idx] -= np.int16(pa[(m,) + idx] * 2 * 2 ** m)
        assert cost(q2, qw) - base == pytest.approx(-2 * pa[(m,) + idx] * ga[(m,) + idx], rel=1e-9, abs=1e-12)
        idw = tuple(int(rng.integers(0, d)) for d in qw.shape)
        j = int(rng.integers(0, wb))
        w2 = qw.copy()
        w2[idw] -= np.int16(pw[(j,) + idw] * 2 * 2 ** j)
        assert cost(qa, w2) - base == pytest.approx(-2 * pw[(j,) + idw] * gw[(j,) + idw], rel=1e-9, abs=1e-12)


@pytest.mark.parametrize("N,H,W,C,Cout,R,S,stride,pad,ab,wb", [(2, 7, 6, 5, 3, 3, 3, 1, 1, 2, 2), (1, 9, 9, 4, 6, 3, 2, 2, 1, 3, 1),
                                                             (2, 5, 5, 8, 2, 1, 1, 2, 0, 1, 4), (1, 8, 7, 3, 5, 5, 5, 1, 2, 2, 2)])
def test_conv_backward_matches_library_autograd(N, H, W, C, Cout, R, S, stride, pad, ab, wb):
    """torch's conv2d differentiated in float64: the per-plane gradients are 2^(m-1) (2^(j-1)) times the gradient with
    respect to the codes."""
    import torch
    qa, qw, g, alpha = _conv_backward_case(N + H + C, N, H, W, C, Cout, R, S, stride, pad, ab, wb)
    a = torch.tensor(qa.transpose(0, 3, 1, 2).astype(np.float64), requires_grad=True)
    w = torch.tensor(qw.transpose(0, 3, 1, 2).astype(np.float64), requires_grad=True)
    out = alpha * torch.nn.functional.conv2d(a, w, stride=stride, padding=pad)
    out.backward(torch.tensor(g.transpose(0, 3, 1, 2).astype(np.float64)))
    da = a.grad.numpy().transpose(0, 2, 3, 1)
    dw = w.grad.numpy().transpose(0, 2, 3, 1)
    ga = oracle.conv_backward_data(g, qw, (H, W), stride, pad, ab, wb, alpha)
    gw = oracle.conv_backward_weights(g, qa, (R, S), stride, pad, ab, wb, alpha)
    for m in range(ab):
        assert np.allclose(ga[m], 2.0 ** m * da, rtol=1e-12, atol=1e-14)
    for j in range(wb):
        assert np.allclose(gw[j], 2.0 ** j * dw, rtol=1e-12, atol=1e-14)


def test_conv_backward_of_a_1x1_convolution_is_the_fc_backward():
    ab, wb = 3, 2
    qa, qw, g, alpha = _conv_backward_case(1, 2, 4, 3, 6, 5, 1, 1, 1, 0, ab, wb)
    ga = oracle.conv_backward_data(g, qw, (4, 3), 1, 0, ab, wb, alpha)
    gw = oracle.conv_backward_weights(g, qa, (1, 1), 1, 0, ab, wb, alpha)
    g2, qa2, qw2 = g.reshape(-1, 5), qa.reshape(-1, 6), qw.reshape(5, 6)
    assert np.allclose(ga.reshape(ab, -1, 6), oracle.fc_backward_data(g2, qw2, ab, wb, alpha), rtol=1e-13, atol=0)
    assert np.allclose(gw.reshape(wb, 5, 6), oracle.fc_backward_weights(g2, qa2, ab, wb, alpha), rtol=1e-13, atol=0)


# ---- Eq. 16 (Section 4.6): the analytic speed-up model -------------------------------------------------------------

def test_eq16_reproduces_the_printed_two_bit_speedup(golden_dir):
    rows = [ln.split() for ln in (golden_dir / "eq16_speedup.txt").read_text().splitlines()
            if ln.strip() and not ln.startswith("#")]
    assert rows
    for n, m, k, gamma, L, printed, allowance in rows:
        s = oracle.eq16_speedup(int(n), int(m), int(k), gamma=float(gamma), reg_len=int(L))
        assert abs(s - float(printed)) <= float(allowance)
        assert abs(oracle.eq16_speedup(int(n), int(m), int(k), gamma=float(gamma), beta=0.0, reg_len=int(L))
                   - float(printed)) > float(allowance)          # the beta term is visible at this precision


def test_eq16_limits_and_shape():
    g, L = 1.91, 64
    # long vectors: the gamma and beta terms vanish against 2*ceil(n/L) per pair -> gamma*L/(2*M*K)
    for m, k in ((1, 1), (2, 2), (3, 5), (8, 8)):
        s = oracle.eq16_speedup(1 << 30, m, k, g, None, L)
        assert math.isclose(s, g * L / (2 * m * k), rel_tol=1e-5)
        # the model only sees the number of plane pairs M*K
        assert oracle.eq16_speedup(8192, m, k) == oracle.eq16_speedup(8192, k, m)
    assert oracle.eq16_speedup(8192, 2, 6) == oracle.eq16_speedup(8192, 3, 4)
    # more pairs never help; one pair of one word: n*gamma / (gamma + 2)
    vals = [oracle.eq16_speedup(8192, b, b) for b in range(1, 9)]
    assert all(a > b for a, b in zip(vals, vals[1:]))
    assert math.isclose(oracle.eq16_speedup(64, 1, 1, g, 0.0, L), 64 * g / (g + 2))
    # a dropped beta term or a floor instead of the ceiling would move these
    assert math.isclose(oracle.eq16_speedup(65, 1, 1, g, None, L), 65 * g / (g + 4))
    assert math.isclose(oracle.eq16_speedup(128, 2, 1, 2.0, 3.0, 64), 128 * 2.0 / (2 * (2.0 + 4) + 3.0))

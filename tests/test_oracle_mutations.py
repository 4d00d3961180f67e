"""Do the pins have teeth?  Each case plants one plausible mistake in a COPY of the oracle's C source
(a dropped term, a wrong sign or index, a flipped tie, a transposed operand), builds it, and requires that
the pin suite fails on it.  The untouched copy must pass.  Everything happens on the CPU."""
import os
import shutil
import subprocess
import sys
from pathlib import Path

import pytest

ROOT = Path(__file__).resolve().parent.parent

MUTATIONS = {
    "tie_towards_zero": ("float tf = (x > 0.0f) ? floorf(v) : ceilf(v) - 1.0f;", "float tf = floorf(v);"),
    "zero_goes_positive": ("float tf = (x > 0.0f) ? floorf(v)", "float tf = (x >= 0.0f) ? floorf(v)"),
    "round_to_nearest_even_grid": ("float v = fmaf(x, inv2s, half);", "float v = fmaf(x, inv2s, half - 0.5f);"),
    "no_clamp_high": ("tf = fminf(fmaxf(tf, 0.0f), amax);", "tf = fmaxf(tf, 0.0f);"),
    "code_offset": ("q[i] = (int16_t)(2 * t - amax);", "q[i] = (int16_t)(2 * t - amax + 1);"),
    "relu_ignored": ("if (relu) x = fmaxf(x, 0.0f);", "(void)relu;"),
    "plane_bit_reversed": ("if ((t >> i) & 1) dst[e / 32]", "if ((t >> (bits - 1 - i)) & 1) dst[e / 32]"),
    "msb_first_in_word": ("|= (uint32_t)1 << (e % 32);", "|= (uint32_t)1 << (31 - e % 32);"),
    "pad_to_one_word": ("return (w + 3) / 4 * 4;", "return w;"),
    "fc_weights_transposed_index": ("(int64_t)qw[n * Kg + k];", "(int64_t)qw[k * Ng + n];"),
    "fc_drops_last_element": ("for (size_t k = 0; k < Kg; ++k)\n                s +=", "for (size_t k = 0; k + 1 < Kg; ++k)\n                s +="),
    "sampled_swaps_row_col": ("const int16_t *a = qa + (size_t)rows[i] * Kg;", "const int16_t *a = qa + (size_t)cols[i] * Kg;"),
    "conv_pad_sign": ("int hi = ho * stride - pad + r;", "int hi = ho * stride + pad + r;"),
    "conv_tap_transposed": ("const int16_t *w = qw + (((size_t)co * R + r) * S + t) * C;", "const int16_t *w = qw + (((size_t)co * S + t) * R + r) * C;"),
    "conv_border_not_skipped": ("if (wi < 0 || wi >= W) continue;", "if (wi < 0) wi = 0; if (wi >= W) wi = W - 1;"),
    "conv_out_dim": ("return (in + 2 * pad - k) / stride + 1;", "return (in + 2 * pad - k + stride - 1) / stride + 1;"),
    "dilation_ignored": ("int hi = ho * stride - pad + r * dil;\n                    if (hi < 0 || hi >= H) continue;", "int hi = ho * stride - pad + r;\n                    if (hi < 0 || hi >= H) continue;"),
    "transposed_scatter_stride": ("int ho = hi * stride - pad + r * dil;", "int ho = hi - pad + r * dil;"),
    "affine_twice_rounded": ("fmaf(y[(size_t)m * Ng + n], gamma[n], beta ? beta[n] : 0.0f);", "y[(size_t)m * Ng + n] * gamma[n] + (beta ? beta[n] : 0.0f);"),
    "backward_data_weight_index_transposed": ("part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qw[n * Kg + k], wb, j);\n                    sum += ldexp(part, m + j - 2);\n                }\n                ga[", "part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qw[(n * Kg + k) % Kg * Ng + (n * Kg + k) / Kg % Ng], wb, j);\n                    sum += ldexp(part, m + j - 2);\n                }\n                ga["),
    "backward_plane_weight_off_by_one": ("sum += ldexp(part, m + j - 2);\n                }\n                gw[", "sum += ldexp(part, m + j - 1);\n                }\n                gw["),
    "backward_drops_alpha": ("part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qa[r * Kg + k], ab, m);\n                    sum += ldexp(part, m + j - 2);\n                }\n                gw[", "part += ((double)g[r * Ng + n]) * plane_of(qa[r * Kg + k], ab, m);\n                    sum += ldexp(part, m + j - 2);\n                }\n                gw["),
    "backward_plane_sign": ("return ((t >> (i - 1)) & 1) ? 1.0 : -1.0;", "return ((t >> (i - 1)) & 1) ? -1.0 : 1.0;"),
    "mbit_lower_planes_not_negated": ("c[(size_t)(m - 1) * n + e] = (m == bits) ? sgn : -sgn;", "c[(size_t)(m - 1) * n + e] = sgn;"),
    "mbit_frequency_uses_2_to_M": ("const float k = (float)((1 << bits) - 1) / (float)(1 << m);", "const float k = (float)(1 << bits) / (float)(1 << m);"),
    "mbit_derivative_not_windowed": ("if (xn >= -1.0 && xn <= 1.0) {", "if (1) {"),
    "mbit_derivative_sine": ("const double d = k * pi * cos(k * pi * xn);", "const double d = k * pi * sin(k * pi * xn);"),
    "mbit_derivative_forgets_r": ("gx[e] = g / (double)r;", "gx[e] = g;"),
    "conv_backward_data_taps_transposed": ("plane_of(qw[(((size_t)co * R + r) * S + s) * C + c], wb, j);", "plane_of(qw[(((size_t)co * S + s) * R + r) * C + c], wb, j);"),
    "conv_backward_weights_drops_alpha": ("part += ((double)alpha * (double)g[(((size_t)n * Ho + ho) * Wo + wo) * Cout + co]) *", "part += ((double)g[(((size_t)n * Ho + ho) * Wo + wo) * Cout + co]) *"),
    "conv_backward_data_ignores_stride": ("const int hi = ho * stride - pad + r, wi = wo * stride - pad + s;\n                            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;\n                            double *dst", "const int hi = ho - pad + r, wi = wo - pad + s;\n                            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;\n                            double *dst"),
    "bitplanes_plane_weight": ("s += ((int64_t)Kg - 2 * differ) * ((int64_t)1 << (i + j));", "s += ((int64_t)Kg - 2 * differ) * ((int64_t)1 << (i * j));"),
    "bitplanes_counts_agreements": ("s += ((int64_t)Kg - 2 * differ) *", "s += (2 * differ - (int64_t)Kg) *"),
    "bitplanes_weight_plane_index": ("const uint32_t *w = w_planes + (n * wb + j) * kw;", "const uint32_t *w = w_planes + (n * wb + (wb - 1 - j)) * kw;"),
    "scale_in_double": ("out[i] = (float)acc[i] * alpha;", "out[i] = (float)((double)acc[i] * (double)alpha * (1.0 + 1e-6));"),
}

# a fast but representative subset of the pins
PIN_ARGS = ["tests/test_oracle_pins.py", "-x", "-q", "-p", "no:cacheprovider"]


def run_pins(pkg_root: Path):
    env = dict(os.environ)
    env["PYTHONPATH"] = f"{pkg_root}{os.pathsep}{ROOT}"
    env["QNN_TEST_ORACLE_ROOT"] = str(pkg_root)
    return subprocess.run([sys.executable, "-m", "pytest", *PIN_ARGS], cwd=ROOT, env=env, capture_output=True,
                          text=True, timeout=600)


def make_copy(tmp: Path, old: str | None, new: str | None) -> Path:
    dst = tmp / "oracle"
    shutil.copytree(ROOT / "oracle", dst, ignore=shutil.ignore_patterns("*.so", "__pycache__"))
    if old is not None:
        src = (dst / "qnn_oracle.c").read_text()
        assert src.count(old) >= 1, f"mutation anchor not found: {old!r}"
        (dst / "qnn_oracle.c").write_text(src.replace(old, new))
    return tmp


def test_unmutated_copy_passes(tmp_path):
    r = run_pins(make_copy(tmp_path, None, None))
    assert r.returncode == 0, r.stdout[-1500:]


@pytest.mark.parametrize("name", sorted(MUTATIONS))
def test_planted_mistake_is_caught(tmp_path, name):
    old, new = MUTATIONS[name]
    r = run_pins(make_copy(tmp_path, old, new))
    assert r.returncode != 0, f"the pins did not notice: {name}"
    assert "CalledProcessError" not in r.stdout + r.stderr, "the mutated source must still compile"
    assert " failed" in r.stdout

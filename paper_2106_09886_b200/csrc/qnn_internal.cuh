// Internal helpers shared by the CUDA translation units of libqnn.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <math.h>
#include "qnn.h"

#define QNN_VERSION_NUMBER 100

static inline bool qnn_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }
static inline bool qnn_bits_ok(int b) { return b >= 1 && b <= 8; }
static inline int64_t qnn_ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
static inline int64_t qnn_row_words_i(int64_t k) { return qnn_ceil_div(qnn_ceil_div(k, 32), 4) * 4; }
static inline int64_t qnn_w_row_words_i(int taps, int c_in) {
    return qnn_ceil_div((int64_t)taps * qnn_ceil_div(c_in, 32), 4) * 4;
}
static inline int qnn_launch_status() { return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_E_CUDA; }

// Unsigned code t in [0, 2^bits - 1] of a real value (odd code q = 2t - (2^bits - 1)).
// inv2s = 1/(2*scale), half = 2^(bits-1), amax = 2^bits - 1, lo = 0 for a fused ReLU else -inf.
// v = x/(2s) + 2^(b-1) with one fused multiply-add; t = floor(v) for x > 0 and ceil(v) - 1 otherwise,
// so that a value half-way between two codes moves away from zero and 0 maps to q = -1.
// ceil(v) - 1 = -floor(-v) - 1 = ~floor(-v): one saturating float->int conversion (round down)
// serves both branches; NaN converts to 0 and ends at t = 0, infinities saturate and are clamped.
__device__ __forceinline__ int qnn_code_t(float x, float inv2s, float half, int amax, float lo) {
    x = fmaxf(x, lo);
    const float v = __fmaf_rn(x, inv2s, half);
    const bool pos = x > 0.0f;
    const int f = __float2int_rd(pos ? v : -v);
    const int t = pos ? f : ~f;
    return min(max(t, 0), amax);
}

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
// Defined in backward.cu: device word shared by all tensor-path kernels (see qnn_tensor_path_status).
unsigned int *qnn_tc_error_word();

// Host-side argument checks of qnn_encode_pack and qnn_bgemm without enqueuing anything (encode.cu, bgemm.cu): the
// composite entry points run both before their first copy or launch.
int qnn_check_encode_pack(const float *x, int64_t rows, int k, int64_t ldx, int bits, float scale, unsigned flags,
                          const uint32_t *planes, const int32_t *rowsum);
int qnn_check_bgemm(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg, float alpha,
                    const float *out, int64_t ldo, const int32_t *acc);

static inline int qnn_launch_status() { return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_E_CUDA; }

// Eq. 8's combine, n*A*B - 2*S, for S = sum_ij 2^(i+j) X_ij <= n*A*B < 2^31: 2*S may reach 2^32, so the subtraction
// is done modulo 2^32 (unsigned) and the result, which always fits, is reinterpreted.
__device__ __forceinline__ int32_t qnn_combine(int32_t n_times_ab, int32_t s) {
    return (int32_t)((uint32_t)n_times_ab - 2u * (uint32_t)s);
}

// Unsigned code t in [0, 2^bits - 1] of a real value (odd code q = 2t - (2^bits - 1)).
// inv2s = 1/(2*scale), half = 2^(bits-1); [lo, hi] is a pre-clamp of x (see qnn_clamp_bounds).
// v = x/(2s) + 2^(b-1) with one fused multiply-add; t = floor(v) for x > 0 and ceil(v) - 1 otherwise,
// so that a value half-way between two codes moves away from zero and 0 maps to q = -1.
// ceil(v) - 1 = -floor(-v) - 1 = ~floor(-v): one float->int conversion (round down) serves both branches.
__device__ __forceinline__ int qnn_code_t(float x, float inv2s, float half, float lo, float hi) {
    x = fminf(fmaxf(x, lo), hi);          // NaN -> lo; no integer clamp is needed afterwards
    const float v = __fmaf_rn(x, inv2s, half);
    const bool pos = x > 0.0f;
    const int f = __float2int_rd(pos ? v : -v);
    return pos ? f : ~f;
}

// The same code without a float->int conversion (those run on the XU pipe, which the contraction's popcounts
// already saturate): returns the bit pattern 0x4B000000 + t, whose low 8 bits are t.  For x <= 0, ceil(v) - 1 is
// floor of the next float below v (bit pattern - 1; v > 0 after the pre-clamp): an integer v loses less than 1, a
// non-integer v cannot fall below floor(v).  floor(y) for 0 <= y < 2^23 is the mantissa of y + 2^23 rounded down.
__device__ __forceinline__ uint32_t qnn_code_bits(float x, float inv2s, float half, float lo, float hi) {
    x = fminf(fmaxf(x, lo), hi);          // NaN -> lo
    const float v = __fmaf_rn(x, inv2s, half);
    const int vb = __float_as_int(v) - ((x > 0.0f) ? 0 : 1);
    return (uint32_t)__float_as_int(__fadd_rd(__int_as_float(vb), 8388608.0f));
}

// Pre-clamp bounds that make the integer clamp of the code unnecessary.  hi = 2^bits * scale * (1 - 2^-10)
// lies between the range end r = (2^bits - 1) * scale and the point where v would reach 2^bits, with a margin
// (2^-11 relative) far above the rounding of inv2s and of the multiply-add: every x in [r, hi] gives
// floor(v) = 2^bits - 1 and every x in [-hi, -r] gives ceil(v) - 1 = 0, exactly the end codes that the
// unclamped formula followed by a clamp of t produces for any |x| >= r.  lo = -hi, or 0 for a fused ReLU
// (also what a NaN input turns into, matching max(NaN, 0) = 0 and NaN -> most negative code).
static inline void qnn_clamp_bounds(int bits, float scale, bool relu, float *lo, float *hi) {
    *hi = (float)(1 << bits) * scale * (1.0f - 0.0009765625f);
    *lo = relu ? 0.0f : -*hi;
}

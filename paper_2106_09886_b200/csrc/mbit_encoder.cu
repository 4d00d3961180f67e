// Training-side form of the encoder: the trigonometric M-bit encoder (Eq. 10) and its derivative (Eq. 12).
// Both are streaming element-wise kernels (bound: HBM; forward reads 4 B and writes 4*bits B per element,
// backward reads 4 + 4*bits B and writes 4 B).
#include "qnn_internal.cuh"
#include "mbit_math.cuh"

namespace {

// sign(sin(pi*y)) without a sine: 0 where y is an integer, +1 where floor(y) is even, -1 where it is odd.
// For |y| < 2^22 the floor and its parity come from one addition of 1.5*2^23: the sum's last mantissa bit is the parity
// of the nearest integer rn, and floor(y) = rn - 1 exactly where rn > y.  Larger |y| (and NaN) take the plain route.
__device__ __forceinline__ float sign_sin_pi(float y) {
    if (fabsf(y) < 4194304.0f) {
        const float t = __fadd_rn(y, 12582912.0f);
        const float rn = __fadd_rn(t, -12582912.0f);
        if (rn == y) return 0.0f;                                  // an exact zero crossing
        const bool odd = ((__float_as_uint(t) & 1u) != 0u) != (rn > y);
        return odd ? -1.0f : 1.0f;
    }
    const float fl = floorf(y);
    if (!(fabsf(y) < INFINITY) || fl == y) return 0.0f;          // NaN, infinity, or an integer
    const float h = __fmul_rn(fl, 0.5f);
    return (floorf(h) == h) ? 1.0f : -1.0f;
}

// One element of Eq. 10: plane m-1 of element e is written to cm[m-1].
template <int BITS>
__device__ __forceinline__ void mbit_forward_elem(float x, float r, float (&cm)[BITS]) {
    const float xn = __fdiv_rn(x, r);
#pragma unroll
    for (int m = 1; m <= BITS; ++m) {
        const float k = (float)((1 << BITS) - 1) / (float)(1 << m);       // exact in binary32
        const float s = sign_sin_pi(__fmul_rn(k, xn));
        cm[m - 1] = (m == BITS) ? s : -s;
    }
}

// VEC = 4: n is a multiple of 4 and every pointer is 16-byte aligned, so each thread moves float4s; VEC = 1 otherwise.
template <int BITS, int VEC>
__global__ void __launch_bounds__(256) mbit_forward_kernel(const float *__restrict__ x, size_t n, float r,
                                                          float *__restrict__ c) {
    const size_t nv = n / VEC;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < nv; e += (size_t)gridDim.x * blockDim.x) {
        if constexpr (VEC == 4) {
            const float4 xv = __ldcs(reinterpret_cast<const float4 *>(x) + e);
            float c0[BITS], c1[BITS], c2[BITS], c3[BITS];
            mbit_forward_elem<BITS>(xv.x, r, c0);
            mbit_forward_elem<BITS>(xv.y, r, c1);
            mbit_forward_elem<BITS>(xv.z, r, c2);
            mbit_forward_elem<BITS>(xv.w, r, c3);
#pragma unroll
            for (int m = 0; m < BITS; ++m)
                __stcs(reinterpret_cast<float4 *>(c + (size_t)m * n) + e, make_float4(c0[m], c1[m], c2[m], c3[m]));
        } else {
            float c0[BITS];
            mbit_forward_elem<BITS>(__ldcs(x + e), r, c0);
#pragma unroll
            for (int m = 0; m < BITS; ++m) __stcs(c + (size_t)m * n + e, c0[m]);
        }
    }
}

template <int BITS, int VEC>
__global__ void __launch_bounds__(256) mbit_backward_kernel(const float *__restrict__ x, const float *__restrict__ gc,
                                                           size_t n, float r, float *__restrict__ gx) {
    const size_t nv = n / VEC;
    for (size_t e = (size_t)blockIdx.x * blockDim.x + threadIdx.x; e < nv; e += (size_t)gridDim.x * blockDim.x) {
        if constexpr (VEC == 4) {
            const float4 xv = __ldcs(reinterpret_cast<const float4 *>(x) + e);
            float g0[BITS], g1[BITS], g2[BITS], g3[BITS];
#pragma unroll
            for (int m = 0; m < BITS; ++m) {
                const float4 gv = __ldcs(reinterpret_cast<const float4 *>(gc + (size_t)m * n) + e);
                g0[m] = gv.x; g1[m] = gv.y; g2[m] = gv.z; g3[m] = gv.w;
            }
            __stcs(reinterpret_cast<float4 *>(gx) + e,
                   make_float4(mbit_backward_elem<BITS>(xv.x, r, g0), mbit_backward_elem<BITS>(xv.y, r, g1),
                               mbit_backward_elem<BITS>(xv.z, r, g2), mbit_backward_elem<BITS>(xv.w, r, g3)));
        } else {
            float g0[BITS];
#pragma unroll
            for (int m = 0; m < BITS; ++m) g0[m] = __ldcs(gc + (size_t)m * n + e);
            gx[e] = mbit_backward_elem<BITS>(__ldcs(x + e), r, g0);
        }
    }
}

int grid_for_elems(size_t n, int vec) {
    size_t blocks = (n / vec + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    return (int)(blocks < 1 ? 1 : blocks);
}

}  // namespace

#define QNN_BITS_SWITCH(bits, CALL) \
    switch (bits) {                 \
        case 1: CALL(1); break;     \
        case 2: CALL(2); break;     \
        case 3: CALL(3); break;     \
        case 4: CALL(4); break;     \
        case 5: CALL(5); break;     \
        case 6: CALL(6); break;     \
        case 7: CALL(7); break;     \
        default: CALL(8); break;    \
    }

extern "C" int qnn_mbit_encoder_forward(const float *x, size_t n, int bits, float r, float *c, void *stream) {
    if (!x || !c || n == 0 || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (!(r >= 1e-30f) || !(r <= 1e30f)) return QNN_E_SCALE;
    if (!qnn_aligned(x, 4) || !qnn_aligned(c, 4)) return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool v4 = n % 4 == 0 && qnn_aligned(x, 16) && qnn_aligned(c, 16);
#define CALL(B)                                                                      \
    if (v4) mbit_forward_kernel<B, 4><<<grid_for_elems(n, 4), 256, 0, st>>>(x, n, r, c); \
    else mbit_forward_kernel<B, 1><<<grid_for_elems(n, 1), 256, 0, st>>>(x, n, r, c)
    QNN_BITS_SWITCH(bits, CALL)
#undef CALL
    return qnn_launch_status();
}

extern "C" int qnn_mbit_encoder_backward(const float *x, const float *gc, size_t n, int bits, float r, float *gx,
                                         void *stream) {
    if (!x || !gc || !gx || n == 0 || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (!(r >= 1e-30f) || !(r <= 1e30f)) return QNN_E_SCALE;
    if (!qnn_aligned(x, 4) || !qnn_aligned(gc, 4) || !qnn_aligned(gx, 4)) return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool v4 = n % 4 == 0 && qnn_aligned(x, 16) && qnn_aligned(gc, 16) && qnn_aligned(gx, 16);
#define CALL(B)                                                                            \
    if (v4) mbit_backward_kernel<B, 4><<<grid_for_elems(n, 4), 256, 0, st>>>(x, gc, n, r, gx); \
    else mbit_backward_kernel<B, 1><<<grid_for_elems(n, 1), 256, 0, st>>>(x, gc, n, r, gx)
    QNN_BITS_SWITCH(bits, CALL)
#undef CALL
    return qnn_launch_status();
}

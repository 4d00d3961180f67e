// Element arithmetic of the encoder derivative (Eq. 12), shared by the stand-alone backward kernel and the epilogue
// of the backward-data product.
#pragma once
#include <cuda_runtime.h>

// gx = (1/r) * sum_m gm[m-1] * d phi_M^m / d xn at xn = x / r: +-k_m*pi*cos(k_m*pi*xn) inside [-1, 1] (sign + for
// m = M), zero outside; k_m = (2^M - 1) / 2^m is exact in binary32.
template <int BITS>
__device__ __forceinline__ float mbit_backward_elem(float x, float r, const float (&gm)[BITS]) {
    const float pi = 3.14159265358979323846f;
    const float xn = __fdiv_rn(x, r);
    float g = 0.0f;
    if (xn >= -1.0f && xn <= 1.0f) {
#pragma unroll
        for (int m = 1; m <= BITS; ++m) {
            const float k = (float)((1 << BITS) - 1) / (float)(1 << m);
            const float d = __fmul_rn(__fmul_rn(k, pi), cospif(__fmul_rn(k, xn)));   // k*pi*cos(k*pi*xn)
            g = __fmaf_rn(gm[m - 1], (m == BITS) ? d : -d, g);
        }
    }
    return __fdiv_rn(g, r);
}

// The same with gm[m-1] = 2^(m-1) * G for every plane (all planes of one activation share the product G of
// Algorithm 1's backward step) and the number of planes known only at run time.
__device__ __forceinline__ float mbit_backward_shared(float x, float r, float G, int bits) {
    const float pi = 3.14159265358979323846f;
    const float xn = __fdiv_rn(x, r);
    float g = 0.0f;
    if (xn >= -1.0f && xn <= 1.0f) {
        const float A = (float)((1 << bits) - 1);
        for (int m = 1; m <= bits; ++m) {
            const float k = A / (float)(1 << m);
            const float d = __fmul_rn(__fmul_rn(k, pi), cospif(__fmul_rn(k, xn)));
            g = __fmaf_rn(__fmul_rn((float)(1 << (m - 1)), G), (m == bits) ? d : -d, g);
        }
    }
    return __fdiv_rn(g, r);
}

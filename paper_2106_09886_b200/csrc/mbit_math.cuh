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
// Algorithm 1's backward step) and the number of planes known only at run time.  The per-plane constants come
// from mbit_plane_consts: k[m-1] = k_m, kpi[m-1] = fl(k_m * pi), pw[m-1] = +-2^(m-1) with the sign of Eq. 12 folded in
// (negating a factor of a product is exact, so the result equals mbit_backward_elem's bit for bit).
struct MbitPlaneConsts {
    float k[8], kpi[8], pw[8];
};

static inline MbitPlaneConsts mbit_plane_consts(int bits) {
    MbitPlaneConsts c{};
    const float pi = 3.14159265358979323846f;
    for (int m = 1; m <= bits && m <= 8; ++m) {
        c.k[m - 1] = (float)((1 << bits) - 1) / (float)(1 << m);
        c.kpi[m - 1] = c.k[m - 1] * pi;
        c.pw[m - 1] = (m == bits) ? (float)(1 << (m - 1)) : -(float)(1 << (m - 1));
    }
    return c;
}

template <int BITS>
__device__ __forceinline__ float mbit_backward_shared(float x, float r, float G, const MbitPlaneConsts &c) {
    const float xn = __fdiv_rn(x, r);
    float g = 0.0f;
#pragma unroll
    for (int m = 0; m < BITS; ++m) {
        const float d = __fmul_rn(c.kpi[m], cospif(__fmul_rn(c.k[m], xn)));
        g = __fmaf_rn(__fmul_rn(c.pw[m], G), d, g);
    }
    g = (xn >= -1.0f && xn <= 1.0f) ? g : 0.0f;          // a select, not a branch: neighbouring elements interleave
    return __fdiv_rn(g, r);
}

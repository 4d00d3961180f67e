// Convolutions whose whole patch fits one 32-bit word per plane (R*S*C <= 32, e.g. a 3x3 first layer on
// 3 channels: 27 bits).  The plane storage keeps every tap on a word boundary, so the general kernel would
// spend a full word operation per tap on C useful bits.  Here the patch word of an output pixel is assembled on
// the fly, bit (tap*C + c), from the taps' plane words (implicit im2col at bit granularity), and the same is
// done once per CTA for the weights.
//
// Mapping: lane <-> output feature (32 consecutive features per pass), so every store is one coalesced
// 128-byte row segment; a warp takes 32 output pixels at a time, lane L assembles pixel L's ab patch words,
// and the pixels' words are then handed round with shuffles.  Per output: ab*wb xors and as many popcounts, fewer for
// 4 x 4 and 3 x 3 bits (dense_weighted_count).
// Taps outside the image are left as zero bits and corrected with tapsum exactly as in the tiled kernel.
#pragma once
#include "qnn_internal.cuh"

namespace qnn_dense {

constexpr int kThreads = 256;

struct Params {
    const uint32_t *a;
    const uint32_t *w;
    const int32_t *tapsum;   // [Ng][taps]
    int64_t Mg;
    int Ng;
    int a_pitch, w_pitch;
    float alpha;
    const float *ch_gamma, *ch_beta;   // optional per-feature affine after the scale
    float *out;
    int32_t *acc;
    int H, W, C, R, S, stride, pad, Ho, Wo;
};


// sum_ij 2^(i+j) popc(a_i xor w_j) for single-word operands.  The popcount pipe is the binding unit of this kernel
// (one popcount per plane pair and output), so for the widest cases the ab*wb xor words are first compressed across
// PAIRS: words of equal weight 2^(i+j) go through full adders on bit columns (sum keeps the weight, carry doubles it),
// 16 words -> 10 for 4 x 4 bits and 9 -> 7 for 3 x 3 bits, at two three-input logic operations per adder.
__device__ __forceinline__ void dense_fa(uint32_t a, uint32_t b, uint32_t c, uint32_t &sum, uint32_t &carry) {
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(sum) : "r"(a), "r"(b), "r"(c));
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(carry) : "r"(a), "r"(b), "r"(c));
}
template <int AB, int WB>
__device__ __forceinline__ int dense_weighted_count(const uint32_t (&a)[AB], const uint32_t (&w)[WB]) {
    if constexpr (AB == 4 && WB == 4) {
        uint32_t x[4][4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
            for (int j = 0; j < 4; ++j) x[i][j] = a[i] ^ w[j];
        uint32_t s2, c2, s3a, c3a, s3, c3b, s4a, c4a, s4, c4b, s5, c5;
        dense_fa(x[0][2], x[1][1], x[2][0], s2, c2);          // weight 4 -> 4 + 8
        dense_fa(x[0][3], x[1][2], x[2][1], s3a, c3a);        // weight 8 -> 8 + 16
        dense_fa(x[3][0], c2, s3a, s3, c3b);
        dense_fa(x[1][3], x[2][2], x[3][1], s4a, c4a);        // weight 16 -> 16 + 32
        dense_fa(c3a, c3b, s4a, s4, c4b);
        dense_fa(x[2][3], x[3][2], c4a, s5, c5);              // weight 32 -> 32 + 64
        return __popc(x[0][0]) + 2 * (__popc(x[0][1]) + __popc(x[1][0])) + 4 * __popc(s2) + 8 * __popc(s3) +
               16 * __popc(s4) + 32 * (__popc(s5) + __popc(c4b)) + 64 * (__popc(x[3][3]) + __popc(c5));
    } else if constexpr (AB == 3 && WB == 3) {
        uint32_t x[3][3];
#pragma unroll
        for (int i = 0; i < 3; ++i)
#pragma unroll
            for (int j = 0; j < 3; ++j) x[i][j] = a[i] ^ w[j];
        uint32_t s2, c2, s3, c3;
        dense_fa(x[0][2], x[1][1], x[2][0], s2, c2);          // weight 4 -> 4 + 8
        dense_fa(x[1][2], x[2][1], c2, s3, c3);               // weight 8 -> 8 + 16
        return __popc(x[0][0]) + 2 * (__popc(x[0][1]) + __popc(x[1][0])) + 4 * __popc(s2) + 8 * __popc(s3) +
               16 * (__popc(x[2][2]) + __popc(c3));
    } else {
        int s = 0;
#pragma unroll
        for (int i = 0; i < AB; ++i)
#pragma unroll
            for (int j = 0; j < WB; ++j) s += __popc(a[i] ^ w[j]) * (1 << (i + j));
        return s;
    }
}

template <int AB, int WB>
__global__ void __launch_bounds__(kThreads) bconv_dense1_kernel(const Params p) {
    extern __shared__ uint32_t smem_u32[];
    const int taps = p.R * p.S;
    uint32_t *wd_s = smem_u32;                                          // [WB][Ng] dense weight words
    int32_t *ts_s = reinterpret_cast<int32_t *>(smem_u32 + WB * p.Ng);  // [taps][Ng]
    for (int idx = threadIdx.x; idx < WB * p.Ng; idx += kThreads) {
        const int j = idx / p.Ng, n = idx - j * p.Ng;
        const uint32_t *src = p.w + ((int64_t)n * WB + j) * p.w_pitch;
        uint32_t word = 0;
        for (int t = 0; t < taps; ++t) word |= src[t] << (t * p.C);
        wd_s[idx] = word;
    }
    for (int idx = threadIdx.x; idx < taps * p.Ng; idx += kThreads) {
        const int t = idx / p.Ng, n = idx - t * p.Ng;
        ts_s[idx] = p.tapsum[(int64_t)n * taps + t];
    }
    __syncthreads();

    constexpr int AMAX = (1 << AB) - 1, PROD = AMAX * ((1 << WB) - 1);
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kThreads) >> 5;
    const int64_t nbatches = (p.Mg + 31) / 32;
    const int ncb = (p.Ng + 31) / 32;

    for (int64_t batch = warp0; batch < nbatches; batch += nwarps) {
        // ---- lane assembles the patch words of output pixel m = batch*32 + lane
        const int64_t m = batch * 32 + lane;
        uint32_t mine[AB];
#pragma unroll
        for (int i = 0; i < AB; ++i) mine[i] = 0u;
        uint32_t invalid = 0u;                                           // bit t set: tap t lies outside the image
        if (m < p.Mg) {
            const int wo = (int)(m % p.Wo);
            const int ho = (int)((m / p.Wo) % p.Ho);
            const int64_t n_img = m / ((int64_t)p.Wo * p.Ho);
            const int h0 = ho * p.stride - p.pad, w0 = wo * p.stride - p.pad;
            int t = 0;
            for (int r = 0; r < p.R; ++r)
                for (int s = 0; s < p.S; ++s, ++t) {
                    const int hi = h0 + r, wi = w0 + s;
                    if (hi >= 0 && hi < p.H && wi >= 0 && wi < p.W) {
                        const uint32_t *src = p.a + ((n_img * p.H + hi) * p.W + wi) * (int64_t)(AB * p.a_pitch);
#pragma unroll
                        for (int i = 0; i < AB; ++i) mine[i] |= __ldg(src + i * p.a_pitch) << (t * p.C);
                    } else {
                        invalid |= 1u << t;
                    }
                }
        }
        const int rows_here = (int)((p.Mg - batch * 32) < 32 ? (p.Mg - batch * 32) : 32);
        // two blocks of 32 features per pass: the pixel's words, its border mask and the row bookkeeping are
        // fetched once for both
        for (int cb = 0; cb < ncb; cb += 2) {
            const bool two = cb + 1 < ncb;                                // warp-uniform
            int n[2];
            bool n_ok[2], affine[2];
            uint32_t wreg[2][WB];
            float gam[2], bet[2];
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                n[h] = (cb + h) * 32 + lane;
                n_ok[h] = n[h] < p.Ng;
#pragma unroll
                for (int j = 0; j < WB; ++j) wreg[h][j] = n_ok[h] ? wd_s[j * p.Ng + n[h]] : 0u;
                affine[h] = p.ch_gamma != nullptr && n_ok[h];
                gam[h] = affine[h] ? __ldg(p.ch_gamma + n[h]) : 1.0f;
                bet[h] = (affine[h] && p.ch_beta) ? __ldg(p.ch_beta + n[h]) : 0.0f;
            }
            for (int rr = 0; rr < rows_here; ++rr) {
                uint32_t arow[AB];
#pragma unroll
                for (int i = 0; i < AB; ++i) arow[i] = __shfl_sync(0xffffffffu, mine[i], rr);
                int s_acc[2];
                s_acc[0] = dense_weighted_count<AB, WB>(arow, wreg[0]);
                s_acc[1] = two ? dense_weighted_count<AB, WB>(arow, wreg[1]) : 0;
                uint32_t inv = __shfl_sync(0xffffffffu, invalid, rr);
                const int n_valid = (taps - __popc(inv)) * p.C;
                int corr[2] = {0, 0};
                while (inv != 0u) {                                       // warp-uniform: the row is the same for all lanes
                    const int t = __ffs(inv) - 1;
                    inv &= inv - 1u;
#pragma unroll
                    for (int h = 0; h < 2; ++h)
                        if (n_ok[h]) corr[h] += ts_s[t * p.Ng + n[h]];
                }
                const int64_t o_row = (batch * 32 + rr) * (int64_t)p.Ng;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (!n_ok[h]) continue;
                    const int32_t v = qnn_combine(n_valid * PROD, s_acc[h] - AMAX * corr[h]);
                    const int64_t o = o_row + n[h];
                    if (p.acc) p.acc[o] = v;
                    if (p.out) {
                        float y = __fmul_rn(__int2float_rn(v), p.alpha);
                        if (affine[h]) y = __fmaf_rn(y, gam[h], bet[h]);
                        p.out[o] = y;
                    }
                }
            }
        }
    }
}

template <int AB, int WB>
inline int launch_dense1(const Params &p, cudaStream_t st) {
    const size_t smem = ((size_t)WB * p.Ng + (size_t)p.R * p.S * p.Ng) * 4u;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return QNN_E_CUDA;
    const int64_t nbatches = (p.Mg + 31) / 32;
    int64_t blocks = (nbatches + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > (int64_t)sms * 8) blocks = (int64_t)sms * 8;
    bconv_dense1_kernel<AB, WB><<<(int)blocks, kThreads, smem, st>>>(p);
    return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_E_CUDA;
}

// usable when the patch fits one word and the per-CTA tables fit the default shared memory
inline bool dense1_applicable(int ab, int wb, int R, int S, int C, int Cout) {
    return ab <= 4 && wb <= 4 && (int64_t)R * S * C <= 32 && C < 32 &&
           ((int64_t)wb * Cout + (int64_t)R * S * Cout) * 4 <= 40 * 1024;
}

inline int dispatch_dense1(int ab, int wb, const Params &p, cudaStream_t st) {
#define QNN_D(A_, W_) \
    if (ab == A_ && wb == W_) return launch_dense1<A_, W_>(p, st);
    QNN_D(1, 1) QNN_D(1, 2) QNN_D(1, 3) QNN_D(1, 4)
    QNN_D(2, 1) QNN_D(2, 2) QNN_D(2, 3) QNN_D(2, 4)
    QNN_D(3, 1) QNN_D(3, 2) QNN_D(3, 3) QNN_D(3, 4)
    QNN_D(4, 1) QNN_D(4, 2) QNN_D(4, 3) QNN_D(4, 4)
#undef QNN_D
    return QNN_E_ARG;
}

}  // namespace qnn_dense

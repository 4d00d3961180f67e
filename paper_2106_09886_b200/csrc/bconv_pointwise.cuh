// Layers whose whole reduction is at most four 32-bit words per plane (Kg <= 128): 1x1 convolutions on up to 128
// channels (the stride-2 projections of a residual network) and fully-connected layers with short rows.
//
// The tiled kernel counts such a reduction word by word (one popcount per xor word and plane pair: its bit-column
// counters need 8 words of ONE pair).  Here the ab*wb*KW xor words of an output are compressed ACROSS plane pairs
// and word positions instead: words of equal weight 2^(i+j) go through full adders on bit columns (the sum keeps the
// weight, the carry doubles it), lowest weights first, and only what is left is counted.  An adder costs two logic
// operations (64 lanes/clk/SM) and saves one popcount (16 lanes/clk/SM), so with W xor words the two pipes balance at
// W/2 adders, where the budget stops: 3 x 3 bits on 64 channels: 18 xor words -> 9 adders, 9 popcounts; 4 x 4 bits on
// 128 channels: 64 words -> 32 adders, 32 popcounts.
//
// Mapping: lane <-> output feature (32 consecutive features per pass, two passes interleaved), so every store is one
// coalesced 128-byte row segment; a warp takes 32 output rows at a time, their plane words staged in the warp's slice
// of shared memory and read back as broadcasts; the packed weights of all features sit in shared memory per CTA.
// A 1x1 convolution without padding has no border, so no tap correction is needed.
#pragma once
#include "qnn_internal.cuh"

namespace qnn_pointwise {

constexpr int kThreads = 256;

struct Params {
    const uint32_t *a;       // activation planes [rows_in][AB][a_pitch]
    const uint32_t *w;       // packed weights [Ng][WB][w_pitch]
    int64_t Mg;
    int Ng, Kg;
    int a_pitch, w_pitch;
    float alpha;
    float *out;
    int64_t ldo;
    int32_t *acc;
    // optional chaining epilogue (as in the tiled kernel): per-feature affine, then the next layer's encoder
    const float *ch_gamma, *ch_beta;   // y = fma(y, ch_gamma[n], ch_beta[n]) (ch_beta may be NULL); ch_gamma NULL: none
    uint32_t *next_planes;             // [Mg][next_bits][next_kw] or NULL
    int next_bits, next_kw;
    float next_inv2s, next_half, next_lo, next_hi;
    int fb_per_item;         // 32-feature blocks that one work item covers: 2, or 1 for problems with few items
    int conv;                // 0: output row m reads activation row m; 1: row m = (n, ho, wo) reads pixel (n, ho*stride, wo*stride)
    int H, W, Ho, Wo, stride;
};

__device__ __forceinline__ void full_adder(uint32_t a, uint32_t b, uint32_t c, uint32_t &sum, uint32_t &carry) {
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(sum) : "r"(a), "r"(b), "r"(c));
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(carry) : "r"(a), "r"(b), "r"(c));
}

// sum_ij 2^(i+j) sum_k popc(a[i][k] xor w[j][k]).  Every loop below has a compile-time trip count and every index is
// a compile-time constant after unrolling, so the class arrays live in registers and the `if`s vanish.
template <int AB, int WB, int KW>
__device__ __forceinline__ int weighted_count(const uint32_t (&a)[AB][4], const uint32_t (&w)[WB][KW]) {
    constexpr int NCLS = AB + WB - 1 + 6;                       // carries climb a few classes above the highest pair
    constexpr int CAP = 2 * (AB < WB ? AB : WB) * KW + 2;       // more than a class ever holds (own words + carries)
    constexpr int FA_BUDGET = (AB * WB * KW + 1) / 2;           // adders beyond this make the logic pipe the slower one
    uint32_t cls[NCLS][CAP];
    int cnt[NCLS];
    int adders = 0;
#pragma unroll
    for (int d = 0; d < NCLS; ++d) cnt[d] = 0;
#pragma unroll
    for (int i = 0; i < AB; ++i)
#pragma unroll
        for (int j = 0; j < WB; ++j)
#pragma unroll
            for (int k = 0; k < KW; ++k) cls[i + j][cnt[i + j]++] = a[i][k] ^ w[j][k];
    int total = 0;
#pragma unroll
    for (int d = 0; d < NCLS; ++d) {
#pragma unroll
        for (int it = 0; it < CAP; ++it) {
            if (cnt[d] >= 3 && adders < FA_BUDGET) {
                ++adders;
                uint32_t s, c;
                full_adder(cls[d][cnt[d] - 1], cls[d][cnt[d] - 2], cls[d][cnt[d] - 3], s, c);
                cnt[d] -= 2;
                cls[d][cnt[d] - 1] = s;
                if (d + 1 < NCLS) cls[d + 1][cnt[d + 1]++] = c;
            }
        }
#pragma unroll
        for (int e = 0; e < CAP; ++e)
            if (e < cnt[d]) total += __popc(cls[d][e]) * (1 << d);      // multiply-add: runs on the FMA pipe, not the ALU
    }
    return total;
}

// Popcounts that weighted_count issues per output (host side, for the roofline): the same greedy reduction on counts.
inline int weighted_count_popcounts(int ab, int wb, int kw) {
    int cnt[32] = {};
    for (int i = 0; i < ab; ++i)
        for (int j = 0; j < wb; ++j) cnt[i + j] += kw;
    int total = 0, adders = 0;
    const int budget = (ab * wb * kw + 1) / 2;
    for (int d = 0; d < 31; ++d) {
        while (cnt[d] >= 3 && adders < budget) { cnt[d] -= 2; ++cnt[d + 1]; ++adders; }
        total += cnt[d];
    }
    return total;
}

// FUSED: with the chaining epilogue (per-feature affine and / or next-layer encoder); a separate instantiation so that
// the plain kernel keeps its registers (sharing one kernel cost it a third of its occupancy and 20% of its speed).
template <int AB, int WB, int KW, bool FUSED>
__global__ void __launch_bounds__(kThreads) pointwise_kernel(const Params p) {
    extern __shared__ uint4 smem4[];
    constexpr int WARPS = kThreads / 32;
    uint4 *rows_s = smem4;                                                     // [WARPS][32 rows][AB] plane words (4 per plane)
    uint32_t *w_s = reinterpret_cast<uint32_t *>(smem4 + WARPS * 32 * AB);     // [WB][KW][Ng]
    // FUSED: per warp two 32 x 32 matrices of code bytes (one per feature block of the item), 16-byte aligned
    uint8_t *codes_all = reinterpret_cast<uint8_t *>(w_s + ((WB * KW * p.Ng + 3) & ~3));
    for (int idx = threadIdx.x; idx < WB * KW * p.Ng; idx += kThreads) {
        const int n = idx % p.Ng, jk = idx / p.Ng;
        const int j = jk / KW, k = jk - j * KW;
        w_s[idx] = p.w[((int64_t)n * WB + j) * p.w_pitch + k];
    }
    __syncthreads();

    constexpr int AMAX = (1 << AB) - 1, PROD = AMAX * ((1 << WB) - 1);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint4 *mine_s = rows_s + warp * 32 * AB;
    uint8_t *codes_s = codes_all + warp * 2048;
    const int64_t warp0 = (int64_t)blockIdx.x * WARPS + warp;
    const int64_t nwarps = (int64_t)gridDim.x * WARPS;
    const int64_t nbatches = (p.Mg + 31) / 32;
    const int ncb = (p.Ng + 31) / 32;
    const int npairs = (ncb + p.fb_per_item - 1) / p.fb_per_item;
    const int base = p.Kg * PROD;

    // work item = (batch of 32 output rows, one or two 32-feature blocks); a warp walks items warp0, warp0 + nwarps, ...
    int64_t staged = -1;                                                       // batch whose rows this warp's slice holds
    for (int64_t item = warp0; item < nbatches * npairs; item += nwarps) {
        const int64_t batch = item / npairs;
        const int cb = (int)(item - batch * npairs) * p.fb_per_item;
        if (batch != staged) {
            // ---- lane stages the plane words of output row m = batch*32 + lane
            const int64_t m = batch * 32 + lane;
            __syncwarp();                                                      // the previous batch's reads are done
            if (m < p.Mg) {
                int64_t src_row = m;
                if (p.conv) {
                    const int wo = (int)(m % p.Wo);
                    const int ho = (int)((m / p.Wo) % p.Ho);
                    const int64_t n_img = m / ((int64_t)p.Wo * p.Ho);
                    src_row = (n_img * p.H + (int64_t)ho * p.stride) * p.W + (int64_t)wo * p.stride;
                }
                const uint4 *src = reinterpret_cast<const uint4 *>(p.a + src_row * (int64_t)(AB * p.a_pitch));
#pragma unroll
                for (int i = 0; i < AB; ++i) mine_s[lane * AB + i] = __ldg(src + i * (p.a_pitch >> 2));
            }
            __syncwarp();
            staged = batch;
        }
        const int rows_here = (int)((p.Mg - batch * 32) < 32 ? (p.Mg - batch * 32) : 32);
        const bool two = p.fb_per_item == 2 && cb + 1 < ncb;                   // warp-uniform
        int n[2];
        bool n_ok[2];
        uint32_t wreg[2][WB][KW];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            n[h] = (cb + h) * 32 + lane;
            n_ok[h] = n[h] < p.Ng && (h == 0 || two);
#pragma unroll
            for (int j = 0; j < WB; ++j)
#pragma unroll
                for (int k = 0; k < KW; ++k) wreg[h][j][k] = n_ok[h] ? w_s[(j * KW + k) * p.Ng + n[h]] : 0u;
        }
#pragma unroll 2
        for (int rr = 0; rr < rows_here; ++rr) {
            uint32_t arow[AB][4];
#pragma unroll
            for (int i = 0; i < AB; ++i) {
                const uint4 v = mine_s[rr * AB + i];                           // same address in every lane: a broadcast
                arow[i][0] = v.x; arow[i][1] = v.y; arow[i][2] = v.z; arow[i][3] = v.w;
            }
            int s_acc[2];
            s_acc[0] = weighted_count<AB, WB, KW>(arow, wreg[0]);
            s_acc[1] = two ? weighted_count<AB, WB, KW>(arow, wreg[1]) : 0;
            const int64_t row = batch * 32 + rr;
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                if (h == 1 && !two) break;                                     // warp-uniform
                const int32_t v = qnn_combine(base, s_acc[h]);
                float y = __fmul_rn(__int2float_rn(v), p.alpha);
                if (FUSED && p.ch_gamma != nullptr && n_ok[h])
                    y = __fmaf_rn(y, __ldg(p.ch_gamma + n[h]), p.ch_beta ? __ldg(p.ch_beta + n[h]) : 0.0f);
                if (n_ok[h]) {
                    if (p.acc) p.acc[row * p.Ng + n[h]] = v;
                    if (p.out) p.out[row * p.ldo + n[h]] = y;
                }
                if (FUSED && p.next_planes != nullptr) {
                    // Next layer's encoder, first half: the code of this output, one byte, into the warp's code matrix
                    // [block h][row rr][feature lane] (0 beyond Ng, so that padding bits come out as 0)
                    const uint32_t code = n_ok[h] ? qnn_code_bits(y, p.next_inv2s, p.next_half, p.next_lo, p.next_hi) : 0u;
                    codes_s[(h * 32 + rr) * 32 + lane] = (uint8_t)code;
                }
            }
        }
        if (FUSED && p.next_planes != nullptr) {
            // Second half: lane L owns row L of the batch: its 32 code bytes per feature block are one word of each
            // plane, gathered four bytes at a time with one mask and one multiply
            // (((c & (0x01010101 << i)) * (0x10204080 >> i)) >> 28 = the four bits) and a funnel shift.
            __syncwarp();
            if (lane < rows_here) {
                const int64_t row = batch * 32 + lane;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    if (h == 1 && !two) break;
                    const uint4 *src = reinterpret_cast<const uint4 *>(codes_s + (h * 32 + lane) * 32);
                    const uint4 lo4 = src[0], hi4 = src[1];
                    const uint32_t c4[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
                    uint32_t *dst = p.next_planes + (row * p.next_bits) * (int64_t)p.next_kw + (cb + h);
                    const bool clear_pad = cb + h == ncb - 1;                  // the row's last feature block: clear the padding words
                    for (int i = 0; i < p.next_bits; ++i, dst += p.next_kw) {
                        const uint32_t mask = 0x01010101u << i, mul = 0x10204080u >> i;
                        uint32_t word = 0u;
#pragma unroll
                        for (int g = 7; g >= 0; --g) word = __funnelshift_l((c4[g] & mask) * mul, word, 4);
                        *dst = word;
                        if (clear_pad)
                            for (int wz = ncb; wz < p.next_kw; ++wz) dst[wz - (cb + h)] = 0u;
                    }
                }
            }
            __syncwarp();                                                      // before the next item overwrites the matrix
        }
    }
}

inline size_t smem_bytes(int ab, int wb, int kw, int Ng, bool fused = false) {
    const size_t weights = ((size_t)wb * kw * Ng + 3) / 4 * 16;               // rounded up to 16 bytes
    return (size_t)(kThreads / 32) * 32 * ab * 16 + weights + (fused ? (size_t)(kThreads / 32) * 2048 : 0);
}

// usable when a row is at most 4 words per plane and the weights of all features fit the default shared memory
inline bool applicable(int ab, int wb, int Kg, int Ng) {
    if (ab > 4 || wb > 4 || Kg > 128) return false;
    return smem_bytes(ab, wb, (Kg + 31) / 32, Ng, true) <= 48u * 1024u;
}

template <int AB, int WB, int KW>
inline int launch(const Params &p_in, cudaStream_t st) {
    Params p = p_in;
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return QNN_E_CUDA;
    // (32 rows, 64 features) per item and warp; 32 features when that leaves warps without work
    int64_t items = ((p.Mg + 31) / 32) * ((p.Ng + 63) / 64);
    p.fb_per_item = 2;
    if (items < (int64_t)sms * 4 * (kThreads / 32)) {
        p.fb_per_item = 1;
        items = ((p.Mg + 31) / 32) * ((p.Ng + 31) / 32);
    }
    int64_t blocks = (items + kThreads / 32 - 1) / (kThreads / 32);
    if (blocks > (int64_t)sms * 4) blocks = (int64_t)sms * 4;
    if (p.ch_gamma != nullptr || p.next_planes != nullptr)
        pointwise_kernel<AB, WB, KW, true><<<(int)blocks, kThreads, smem_bytes(AB, WB, KW, p.Ng, true), st>>>(p);
    else
        pointwise_kernel<AB, WB, KW, false><<<(int)blocks, kThreads, smem_bytes(AB, WB, KW, p.Ng), st>>>(p);
    return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_E_CUDA;
}

template <int AB>
inline int run_ab(int wb, int kw, const Params &p, cudaStream_t st) {
#define QNN_PW(W_, K_) \
    if (wb == W_ && kw == K_) return launch<AB, W_, K_>(p, st);
    QNN_PW(1, 1) QNN_PW(1, 2) QNN_PW(1, 3) QNN_PW(1, 4)
    QNN_PW(2, 1) QNN_PW(2, 2) QNN_PW(2, 3) QNN_PW(2, 4)
    QNN_PW(3, 1) QNN_PW(3, 2) QNN_PW(3, 3) QNN_PW(3, 4)
    QNN_PW(4, 1) QNN_PW(4, 2) QNN_PW(4, 3) QNN_PW(4, 4)
#undef QNN_PW
    return QNN_E_ARG;
}

// one translation unit per activation width (pointwise_ab<N>.cu) so that the instantiations build in parallel
int run_pointwise_ab1(int wb, int kw, const Params &p, cudaStream_t st);
int run_pointwise_ab2(int wb, int kw, const Params &p, cudaStream_t st);
int run_pointwise_ab3(int wb, int kw, const Params &p, cudaStream_t st);
int run_pointwise_ab4(int wb, int kw, const Params &p, cudaStream_t st);

inline int dispatch(int ab, int wb, const Params &p, cudaStream_t st) {
    const int kw = (p.Kg + 31) / 32;
    switch (ab) {
        case 1: return run_pointwise_ab1(wb, kw, p, st);
        case 2: return run_pointwise_ab2(wb, kw, p, st);
        case 3: return run_pointwise_ab3(wb, kw, p, st);
        case 4: return run_pointwise_ab4(wb, kw, p, st);
        default: return QNN_E_ARG;
    }
}

}  // namespace qnn_pointwise

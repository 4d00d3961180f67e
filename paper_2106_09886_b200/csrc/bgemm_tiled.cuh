// Tiled xor+popcount contraction for ab, wb in 1..8 (FC and implicit-im2col convolution).
//
// Persistent CTAs (two per SM) walk over output tiles; the first stage of the next tile is copied
// while the last stage of the current one is computed and written out.
// CTA tile: BM activation rows x 64 output features, 256 threads, each thread a TM x 4 block of
// outputs (rows ty + 16r, features tx + 16c) for ALL ab*wb plane pairs; TM = 4 (BM = 64) for
// ab <= 2 and TM = 2 (BM = 32) for ab = 3, 4, so that the TM*ab*8 re-coded activation words of a
// group stay in registers while the weight words stream past them.  The reduction runs in
// stages of 16 words (512 elements) per (row, plane), double buffered in shared memory with
// cp.async; the operand words of a stage are re-coded in place before use (see below).
//
// Carry-save contraction.  popcount issues at 16 lanes/clk/SM, 3-input logic at 64, so counting
// every xor word separately is popcount-bound.  Eight xor words x0..x7 of one (output, plane pair)
// are instead compressed with full adders on bit columns (a 7:3 counter: ones, twos, fours) and
// only 4 words are counted: popc(ones) + popc(x7) + 2 popc(twos) + 4 popc(fours).
// Because xor distributes over the operands, the sum output of an adder whose inputs are
// x_p ^ x_q ^ x_r equals (a_p^a_q^a_r) ^ (w_p^w_q^w_r): the operand-side xors are computed ONCE
// per staged word (not per output), so shared memory holds, per group of 8 words,
//   T = [a0, a1, a0^a1^a2, a3, a4, a3^a4^a5, a0^...^a6, a7]
// and the per-output work is 8 xors + 5 three-input logic ops + 4 popcounts + 4 multiply-adds.
#pragma once
#include "qnn_internal.cuh"

namespace qnn_tiled {

constexpr int kBN = 64, kThreads = 256;
// default rows per thread: 4 (BM = 64) for ab <= 2, 2 (BM = 32) for ab = 3, 4, 1 (BM = 16) for ab >= 5 (so that
// TM*ab*8 operand words never exceed 64 registers); ab <= 2 also has a TM = 2
// instantiation, used when halving the tile fills the SMs' CTA slots more evenly, and ab = 4 a TM = 1 one that runs
// three CTAs per SM (fully-connected layers and 3x3 convolutions with 9-word groups, see launch_tiled).  One-bit
// activations (32 operand registers at TM = 4) also run three CTAs per SM: with a single plane the staging, re-coding
// and barrier of a stage weigh twice what they do at two bits, and a third CTA hides them (+3 to +6%).
template <int AB> struct TileM { static constexpr int TM = (AB <= 2) ? 4 : (AB <= 4 ? 2 : 1); };
constexpr int kStageChunks = 2;                   // groups of 8 words per stage
constexpr int kStageWords = 8 * kStageChunks;     // words per (row, plane) per stage

struct Params {
    const uint32_t *a;
    const uint32_t *w;
    const int32_t *tapsum;   // conv only: [Ng][taps]
    int64_t Mg;
    int Ng;
    int a_pitch, w_pitch;    // words per (row|pixel, plane) and per (feature, plane)
    int kwords;              // words to contract per plane: FC = a_pitch, conv = taps*cw
    int nfull;               // groups of 8 words that go through the 7:3 counters
    int ntail;               // 0..3 words after them, counted one by one
    int nstages;             // ceil((nfull + (ntail > 0)) / 2)
    int tiles_m, ntiles;     // tile t covers rows (t % tiles_m)*BM.. and features (t / tiles_m)*64..
    int n_elems;             // FC: Kg (true reduction length)
    float alpha;
    float *out;
    int64_t ldo;
    int32_t *acc;
    // convolution geometry
    int H, W, C, R, S, stride, pad, Ho, Wo, cw, piece;   // piece = words per copy (4, 2 or 1)
    int dil, transposed;                                  // KIND 2 only: dilation (>= 1), transposed flag
    uint32_t cw_magic, s_magic;                           // x / d == (x * magic) >> 20 for the ranges used
    // exact division of any numerator below 2^31 by Wo, Ho*Wo and tiles_m: n / d == (n * magic) >> shift in 64 bits
    // (see set_fastdiv).  fast_pix = 0: rows or images beyond that range, use plain 64-bit division.
    uint32_t wo_magic, howo_magic, tm_magic;
    int wo_shift, howo_shift, tm_shift, fast_pix;
    // optional per-feature affine applied after the scale: y = fma(y, ch_gamma[n], ch_beta[n]) (ch_beta may be NULL)
    const float *ch_gamma, *ch_beta;
    // fused next-layer encoder (optional): planes of the fp32 result, rows = output rows, k = Ng
    uint32_t *next_planes;   // [Mg][next_bits][next_kw] or NULL
    int next_bits, next_kw;
    float next_inv2s, next_half, next_lo, next_hi;
};

// Splits kwords into full 8-word groups and a short tail: a remainder of 4..7 words is cheaper as one
// more zero-padded group (4 popcounts) than word by word.
inline void set_k_split(Params &p) {
    p.nfull = p.kwords / 8;
    p.ntail = p.kwords % 8;
    if (p.ntail >= 4) { ++p.nfull; p.ntail = 0; }
    p.nstages = (p.nfull + (p.ntail > 0 ? 1 : 0) + kStageChunks - 1) / kStageChunks;
}

// Division by an invariant divisor d (1 <= d < 2^31) of numerators n < 2^31: with k = 31 + ceil(log2 d) and
// magic = ceil(2^k / d) (< 2^32), floor(n * magic / 2^k) = floor(n / d) exactly (the error n * (magic*d - 2^k) / (d * 2^k)
// stays below 1/d).  The tile bookkeeping divides row indices by the output width and by the pixels per image for
// every tile; the generic 64-bit division costs over a hundred instructions each.
inline void set_fastdiv(uint32_t d, uint32_t &magic, int &shift) {
    int lg = 0;
    while ((1ull << lg) < d) ++lg;
    shift = 31 + lg;
    magic = (uint32_t)(((1ull << shift) + d - 1) / d);
}
__device__ __forceinline__ uint32_t fastdiv(uint32_t n, uint32_t magic, int shift) {
    return (uint32_t)(((uint64_t)n * magic) >> shift);
}

__device__ __forceinline__ uint32_t lop3_xor3(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t lop3_maj(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
// carry of the full adder with inputs (u, v, z) given u, v and the adder's SUM s = u^v^z
__device__ __forceinline__ uint32_t lop3_carry_from_sum(uint32_t u, uint32_t v, uint32_t s) {
    uint32_t d;
    asm("lop3.b32 %0, %1, %2, %3, 0xD4;" : "=r"(d) : "r"(u), "r"(v), "r"(s));
    return d;
}

// Input coordinate read by tap index r of an output whose base coordinate is `base`, along one axis.
// Forward convolution: base = o*stride - pad, coordinate base + r*dil.  Transposed convolution: base = o + pad,
// the tap contributes only where (base - r*dil) is a non-negative multiple of the stride, coordinate = quotient.
__device__ __forceinline__ bool tap_coord(const Params &p, int base, int r, int limit, int &pos) {
    if (!p.transposed) {
        pos = base + r * p.dil;
        return pos >= 0 && pos < limit;
    }
    const int t = base - r * p.dil;
    pos = (t >= 0) ? t / p.stride : 0;
    return t >= 0 && pos * p.stride == t && pos < limit;
}

__device__ __forceinline__ void cp_async(uint32_t dst_smem, const void *src, int bytes_total, bool valid) {
    // 16-, 8- or 4-byte asynchronous copy; an invalid source is replaced by zeros (src-size 0)
    const int n = valid ? bytes_total : 0;
    if (bytes_total == 16)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
    else if (bytes_total == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst_smem), "l"(src), "r"(n) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_group 0;" ::: "memory"); }

// One (output, plane pair) over 8 re-coded words: returns nothing, adds the weighted count.
// `shift` = i + j is a compile-time constant after unrolling.
__device__ __forceinline__ void pair8(const uint32_t (&ta)[8], const uint32_t (&tw)[8], const int shift, int &acc) {
    const uint32_t u = ta[0] ^ tw[0], v = ta[1] ^ tw[1], s1 = ta[2] ^ tw[2];
    const uint32_t c1 = lop3_carry_from_sum(u, v, s1);
    const uint32_t u2 = ta[3] ^ tw[3], v2 = ta[4] ^ tw[4], s2 = ta[5] ^ tw[5];
    const uint32_t c2 = lop3_carry_from_sum(u2, v2, s2);
    const uint32_t ones = ta[6] ^ tw[6];                       // x0^...^x6 = s1^s2^x6
    const uint32_t c3 = lop3_carry_from_sum(s1, s2, ones);     // carry of (s1, s2, x6)
    const uint32_t twos = lop3_xor3(c1, c2, c3), fours = lop3_maj(c1, c2, c3);
    const uint32_t x7 = ta[7] ^ tw[7];
    acc += __popc(ones) * (1 << shift);
    acc += __popc(x7) * (1 << shift);
    acc += __popc(twos) * (2 << shift);
    acc += __popc(fours) * (4 << shift);
}

// Nine re-coded words [x0, x1, x0^x1^x2, x3, x4, x3^x4^x5, x6, x7, x6^x7^x8] of one (output, plane pair):
// three 3:2 counters, a fourth on their sums and one on their carries: 12 xors/logic ops + 4 three-input
// ops, 4 popcounts (ones, two words of weight 2, fours).  Used where the reduction is a multiple of 9 words
// (3x3 convolutions, one group = one channel word of all nine taps), which then has no tail.
__device__ __forceinline__ void pair9(const uint32_t (&ta)[9], const uint32_t (&tw)[9], const int shift, int &acc) {
    const uint32_t u1 = ta[0] ^ tw[0], v1 = ta[1] ^ tw[1], s1 = ta[2] ^ tw[2];
    const uint32_t c1 = lop3_carry_from_sum(u1, v1, s1);
    const uint32_t u2 = ta[3] ^ tw[3], v2 = ta[4] ^ tw[4], s2 = ta[5] ^ tw[5];
    const uint32_t c2 = lop3_carry_from_sum(u2, v2, s2);
    const uint32_t u3 = ta[6] ^ tw[6], v3 = ta[7] ^ tw[7], s3 = ta[8] ^ tw[8];
    const uint32_t c3 = lop3_carry_from_sum(u3, v3, s3);
    const uint32_t ones = lop3_xor3(s1, s2, s3), c4 = lop3_maj(s1, s2, s3);
    const uint32_t twos = lop3_xor3(c1, c2, c3), fours = lop3_maj(c1, c2, c3);
    acc += __popc(ones) * (1 << shift);
    acc += __popc(twos) * (2 << shift);
    acc += __popc(c4) * (2 << shift);
    acc += __popc(fours) * (4 << shift);
}

// KIND: 0 = fully-connected operand, 1 = convolution gather, 3 = 3x3 convolution gather with 9-word groups, 2 = dilated / transposed convolution gather (its
// own instantiation: carrying that index arithmetic in the plain convolution cost it up to 15%).
template <int AB, int WB, int KIND, int TM, bool FUSED>
__global__ void __launch_bounds__(kThreads, ((TM == 1 && AB == 4 && (KIND == 0 || KIND == 3)) || (AB == 1 && KIND != 2)) ? 3 : 2) bgemm_tiled_kernel(const Params p) {
    constexpr bool CONV = KIND != 0, GENERAL = KIND == 2, G9 = KIND == 3;
    // multiply-shift division in the tile bookkeeping: convolutions with ab <= 4 only (the fully-connected kernels
    // divide once per tile, and both they and the 16-row-tile kernels for ab >= 5 ran 2-5% slower with it compiled
    // in, through register-allocation side effects)
    constexpr bool FASTDIV = CONV && AB <= 4;
    constexpr int kBM = 16 * TM;
    constexpr int A_UNITS = kBM * AB * kStageChunks;      // (row, plane, group) units per stage
    constexpr int W_UNITS = kBN * WB * kStageChunks;
    constexpr int A_VEC = kStageChunks * 2 * AB * kBM;    // uint4 per stage, A region
    constexpr int W_VEC = kStageChunks * 2 * WB * kBN;
    // G9 keeps the ninth word of every group in a separate uint32 region [group slot][plane][row] per operand
    constexpr int A_EXT = kStageChunks * AB * kBM, W_EXT = kStageChunks * WB * kBN;          // words
    constexpr int BUF_VEC = A_VEC + W_VEC + (G9 ? (A_EXT + W_EXT + 3) / 4 : 0);             // uint4 per buffer
    extern __shared__ uint4 smem[];                       // [2 buffers][BUF_VEC]
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const uint32_t smem_base = (uint32_t)__cvta_generic_to_shared(smem);
    // staging: unit u = tid + 256*q  ->  row = tid % BM (A) or tid % 64 (W) for every q; the A operand has
    // at most one unit per thread and stage, the W operand at most four.
    constexpr int W_Q = (W_UNITS + kThreads - 1) / kThreads;   // W units per thread and stage (1..4)
    static_assert(A_UNITS <= kThreads && W_Q <= 4, "staging map");
    const int srow = tid % kBM, wrow = tid % kBN;
    const int ngroups = p.nfull + (p.ntail > 0 ? 1 : 0);
    const bool a_unit = tid < A_UNITS;
    const int a_plane = (tid % (kBM * AB)) / kBM, a_ch = tid / (kBM * AB);
    const uint32_t a_dst0 = (uint32_t)(((a_ch * 2 * AB + a_plane) * kBM + srow) * 16);   // + g*AB*BM*16

    // Per-tile source bookkeeping of this thread's units.
    struct TileSrc {
        const uint32_t *a;      // FC: start of this thread's (row, plane) words; conv: unused
        const uint32_t *w[W_Q]; // start of this thread's (feature, plane) words, per unit
        int64_t pixbase;        // conv: n*H*W of the row's image
        int h0, w0;             // conv: top-left input coordinate of the row's window
        bool a_ok, w_ok;
        int tile_n;             // feature tile (selects the weights)
    };
    auto prep_tile = [&](int tile) {
        TileSrc t;
        const int tile_n = FASTDIV ? (int)fastdiv((uint32_t)tile, p.tm_magic, p.tm_shift) : tile / p.tiles_m;
        const int64_t m0 = (int64_t)(tile - tile_n * p.tiles_m) * kBM;
        const int n0 = tile_n * kBN;
        const int64_t am = m0 + srow;
        t.tile_n = tile_n;
        t.a_ok = a_unit && am < p.Mg;
        t.w_ok = (n0 + wrow) < p.Ng;
        t.a = p.a + ((int64_t)(t.a_ok ? am : 0) * AB + a_plane) * p.a_pitch;
        t.pixbase = 0; t.h0 = 0; t.w0 = 0;
        if (CONV) {
            const int64_t mm = t.a_ok ? am : 0;
            int wo, ho;
            int64_t n;
            if (FASTDIV && p.fast_pix) {
                const uint32_t m32 = (uint32_t)mm;
                const uint32_t q = fastdiv(m32, p.wo_magic, p.wo_shift), img = fastdiv(m32, p.howo_magic, p.howo_shift);
                wo = (int)(m32 - q * (uint32_t)p.Wo);
                ho = (int)(q - img * (uint32_t)p.Ho);
                n = img;
            } else {
                wo = (int)(mm % p.Wo);
                ho = (int)((mm / p.Wo) % p.Ho);
                n = mm / ((int64_t)p.Wo * p.Ho);
            }
            t.h0 = (GENERAL && p.transposed) ? ho + p.pad : ho * p.stride - p.pad;
            t.w0 = (GENERAL && p.transposed) ? wo + p.pad : wo * p.stride - p.pad;
            t.pixbase = n * p.H * p.W;
        }
#pragma unroll
        for (int q = 0; q < W_Q; ++q) {
            const int u = tid + q * kThreads;
            const int plane = (u % (kBN * WB)) / kBN;
            t.w[q] = p.w + ((int64_t)(t.w_ok ? n0 + wrow : 0) * WB + plane) * p.w_pitch;
        }
        return t;
    };

    // 9-word-group kernels keep the weights resident: their tiles have one or two stages, so stage s of every tile
    // lands in the same buffer (two stages) or the buffers alternate (one stage), and a CTA walks many row tiles of one
    // feature tile.  w_tag[buf] records which (feature tile, stage) weights buffer `buf` holds, already re-coded; a
    // stage whose weights are there copies and re-codes only its activations (two thirds of a stage's copies are
    // weights).  The tags are the same in every thread of the CTA.
    int w_tag0 = -1, w_tag1 = -1;
    bool w_fresh0 = false, w_fresh1 = false;   // weights copied for the pending stage of that buffer: re-code them
    // Copies stage `stage` of the tile described by `t` into buffer `buf` (asynchronously; one commit group).
    auto issue_stage = [&](const TileSrc &t, int stage, int buf) {
        const uint32_t a_smem = smem_base + (uint32_t)buf * BUF_VEC * 16u;
        const uint32_t w_smem = a_smem + A_VEC * 16u;
        if constexpr (G9) {
            // group gi = channel word gi of all nine taps: nine 4-byte copies per (row, plane) unit
            const uint32_t a_ext = a_smem + (uint32_t)(A_VEC + W_VEC) * 16u, w_ext = a_ext + (uint32_t)A_EXT * 4u;
            if (a_unit) {
                const int gi = stage * kStageChunks + a_ch;
                if (gi < p.nfull) {
                    // a 3 x 3 window: tap = 3*r + sx at compile time; the window's top-left word once, the taps as
                    // row / pixel steps from it, the border tests once per row and column of the window
                    const int pix_step = AB * p.a_pitch;
                    const int64_t row_step = (int64_t)p.W * pix_step;
                    const uint32_t *base = p.a + ((t.pixbase + (int64_t)t.h0 * p.W + t.w0) * AB + a_plane) * p.a_pitch + gi;
                    bool okh[3], okw[3];
#pragma unroll
                    for (int d = 0; d < 3; ++d) {
                        okh[d] = t.a_ok && t.h0 + d >= 0 && t.h0 + d < p.H;
                        okw[d] = t.w0 + d >= 0 && t.w0 + d < p.W;
                    }
#pragma unroll
                    for (int tap = 0; tap < 9; ++tap) {
                        constexpr int kR[9] = {0, 0, 0, 1, 1, 1, 2, 2, 2}, kS[9] = {0, 1, 2, 0, 1, 2, 0, 1, 2};
                        const bool ok = okh[kR[tap]] && okw[kS[tap]];
                        const uint32_t *src = base + kR[tap] * row_step + kS[tap] * pix_step;
                        const uint32_t dst = tap < 8 ? a_smem + a_dst0 + (uint32_t)((tap >> 2) * AB * kBM * 16 + (tap & 3) * 4)
                                                     : a_ext + (uint32_t)(((a_ch * AB + a_plane) * kBM + srow) * 4);
                        cp_async(dst, ok ? (const void *)src : (const void *)p.a, 4, ok);
                    }
                }
            }
            const int tag = t.tile_n * 2 + stage;
            const bool fresh = (buf ? w_tag1 : w_tag0) != tag;
            if (buf) { w_tag1 = tag; w_fresh1 = fresh; } else { w_tag0 = tag; w_fresh0 = fresh; }
#pragma unroll
            for (int q = 0; q < W_Q; ++q) {
                const int u = tid + q * kThreads;
                if ((W_UNITS % kThreads) != 0 && u >= W_UNITS) break;
                if (!fresh) break;                                           // these weights are resident
                const int rp = u % (kBN * WB), ch = u / (kBN * WB);
                const int plane = rp / kBN;
                const int gi = stage * kStageChunks + ch;
                if (gi >= p.nfull) continue;
#pragma unroll
                for (int tap = 0; tap < 9; ++tap) {
                    const uint32_t dst = tap < 8 ? w_smem + (uint32_t)((((ch * 2 + (tap >> 2)) * WB + plane) * kBN + wrow) * 16 + (tap & 3) * 4)
                                                 : w_ext + (uint32_t)(((ch * WB + plane) * kBN + wrow) * 4);
                    cp_async(dst, t.w_ok ? (const void *)(t.w[q] + tap * p.cw + gi) : (const void *)p.w, 4, t.w_ok);
                }
            }
            cp_async_commit();
            return;
        }
        if (a_unit) {
            const int gi = stage * kStageChunks + a_ch;
            if (gi < ngroups) {
                const int kw0 = gi * 8;
                const bool full = gi < p.nfull;              // the tail group only needs its first 4 words
                if (!CONV) {
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (g == 1 && !full) break;
                        const int kw = kw0 + 4 * g;
                        const bool ok = t.a_ok && kw < p.kwords;
                        cp_async(a_smem + a_dst0 + (uint32_t)(g * AB * kBM * 16), ok ? (const void *)(t.a + kw) : (const void *)p.a,
                                 16, ok);
                    }
                } else {
                    const int piece = p.piece;
                    const int nwords = full ? 8 : 4;
                    for (int off = 0; off < nwords; off += piece) {
                        const int kw = kw0 + off;
                        const int tap = (int)(((uint32_t)kw * p.cw_magic) >> 20);
                        const int cword = kw - tap * p.cw;
                        const int r = (int)(((uint32_t)tap * p.s_magic) >> 20), s = tap - r * p.S;
                        int hi = t.h0 + r, wi = t.w0 + s;
                        bool ok = t.a_ok && kw < p.kwords && hi >= 0 && hi < p.H && wi >= 0 && wi < p.W;
                        if (GENERAL) {
                            const bool okh = tap_coord(p, t.h0, r, p.H, hi), okw = tap_coord(p, t.w0, s, p.W, wi);
                            ok = t.a_ok && kw < p.kwords && okh && okw;
                        }
                        const uint32_t *src =
                            p.a + ((t.pixbase + (int64_t)hi * p.W + wi) * AB + a_plane) * p.a_pitch + cword;
                        const uint32_t dst = a_smem + a_dst0 + (uint32_t)((off >> 2) * AB * kBM * 16) + (uint32_t)(off & 3) * 4u;
                        cp_async(dst, ok ? (const void *)src : (const void *)p.a, piece * 4, ok);
                    }
                }
            }
        }
#pragma unroll
        for (int q = 0; q < (W_UNITS + kThreads - 1) / kThreads; ++q) {
            const int u = tid + q * kThreads;
            if ((W_UNITS % kThreads) != 0 && u >= W_UNITS) break;
            const int rp = u % (kBN * WB), ch = u / (kBN * WB);
            const int plane = rp / kBN;
            const int gi = stage * kStageChunks + ch;
            if (gi >= ngroups) continue;
            const int kw0 = gi * 8;
            const bool full = gi < p.nfull;
#pragma unroll
            for (int g = 0; g < 2; ++g) {
                if (g == 1 && !full) break;
                const int kw = kw0 + 4 * g;
                const bool ok = t.w_ok && kw < p.kwords && kw < p.w_pitch;
                const uint32_t dst = w_smem + (uint32_t)((((ch * 2 + g) * WB + plane) * kBN + wrow) * 16);
                cp_async(dst, ok ? (const void *)(t.w[q] + kw) : (const void *)p.w, 16, ok);
            }
        }
        cp_async_commit();
    };

    // re-code the full groups this thread copied: [x0..x7] -> [x0, x1, x0^x1^x2, x3, x4, x3^x4^x5, x0^..^x6, x7]
    auto recode_stage = [&](int stage, int buf) {
        uint4 *a_s = smem + (size_t)buf * BUF_VEC;
        uint4 *w_s = a_s + A_VEC;
        auto recode = [](uint4 *lo, uint4 *hi) {
            uint4 x = *lo, y = *hi;
            const uint32_t t2 = lop3_xor3(x.x, x.y, x.z);
            const uint32_t t5 = lop3_xor3(x.w, y.x, y.y);
            const uint32_t t6 = lop3_xor3(t2, t5, y.z);
            *lo = make_uint4(x.x, x.y, t2, x.w);
            *hi = make_uint4(y.x, t5, t6, y.w);
        };
        if constexpr (G9) {
            // [x0..x8] -> [x0, x1, x0^x1^x2, x3, x4, x3^x4^x5, x6, x7, x6^x7^x8]
            uint32_t *a_e = reinterpret_cast<uint32_t *>(a_s + A_VEC + W_VEC), *w_e = a_e + A_EXT;
            auto recode9 = [](uint4 *lo, uint4 *hi, uint32_t *ext) {
                uint4 x = *lo, y = *hi;
                const uint32_t x8 = *ext;
                *lo = make_uint4(x.x, x.y, lop3_xor3(x.x, x.y, x.z), x.w);
                *hi = make_uint4(y.x, lop3_xor3(x.w, y.x, y.y), y.z, y.w);
                *ext = lop3_xor3(y.z, y.w, x8);
            };
            if (a_unit && stage * kStageChunks + a_ch < p.nfull)
                recode9(a_s + ((a_ch * 2 + 0) * AB + a_plane) * kBM + srow, a_s + ((a_ch * 2 + 1) * AB + a_plane) * kBM + srow,
                        a_e + (a_ch * AB + a_plane) * kBM + srow);
#pragma unroll
            for (int q = 0; q < W_Q; ++q) {
                const int u = tid + q * kThreads;
                if ((W_UNITS % kThreads) != 0 && u >= W_UNITS) break;
                if (!(buf ? w_fresh1 : w_fresh0)) break;                     // resident weights are already re-coded
                const int rp = u % (kBN * WB), ch = u / (kBN * WB);
                const int plane = rp / kBN;
                if (stage * kStageChunks + ch >= p.nfull) continue;
                recode9(w_s + ((ch * 2 + 0) * WB + plane) * kBN + wrow, w_s + ((ch * 2 + 1) * WB + plane) * kBN + wrow,
                        w_e + (ch * WB + plane) * kBN + wrow);
            }
            return;
        }
        if (a_unit && stage * kStageChunks + a_ch < p.nfull)
            recode(a_s + ((a_ch * 2 + 0) * AB + a_plane) * kBM + srow, a_s + ((a_ch * 2 + 1) * AB + a_plane) * kBM + srow);
#pragma unroll
        for (int q = 0; q < (W_UNITS + kThreads - 1) / kThreads; ++q) {
            const int u = tid + q * kThreads;
            if ((W_UNITS % kThreads) != 0 && u >= W_UNITS) break;
            const int rp = u % (kBN * WB), ch = u / (kBN * WB);
            const int plane = rp / kBN;
            if (stage * kStageChunks + ch >= p.nfull) continue;
            recode(w_s + ((ch * 2 + 0) * WB + plane) * kBN + wrow, w_s + ((ch * 2 + 1) * WB + plane) * kBN + wrow);
        }
    };

    // Chaining epilogue, second half (see the first half in the epilogue below): thread (row, w) owns word w (32 features)
    // of tile row `row`: it reads the 32 code bytes and moves bit i of each byte into plane i's word four bytes at a time
    // with one mask and one multiply (((c & (0x01010101 << i)) * (0x10204080 >> i)) >> 28 = the four bits; the partial
    // products land on distinct bits), appended by a funnel shift.  Replaces one warp ballot per plane and 16 features.
    // It runs AFTER the first stage barrier of the CTA's next tile (or a barrier of its own after the last tile), so a
    // tile costs no barrier of its own for it; the code matrix is double-buffered, which keeps the next epilogue's
    // writes away from these reads.
    int64_t pend_m0 = -1;                              // tile whose codes wait to be packed (-1: none); same in all threads
    int pend_n0 = 0, pend_buf = 0;
    auto pack_pending = [&]() {
        // one (row, word of the tile, plane) per thread: 2 * kBM units per plane, kThreads / (2 * kBM) planes at a time
        constexpr int PLANES_AT_ONCE = kThreads / (2 * kBM);
        const int unit = tid % (2 * kBM);
        const int row = unit >> 1, wsel = unit & 1;
        const int64_t m = pend_m0 + row;
        if (m < p.Mg) {
            const uint4 *src = reinterpret_cast<const uint4 *>(reinterpret_cast<const uint8_t *>(smem + 2 * BUF_VEC) +
                                                               pend_buf * (kBM * kBN)) + row * 4 + wsel * 2;
            const uint4 lo4 = src[0], hi4 = src[1];
            const uint32_t c4[8] = {lo4.x, lo4.y, lo4.z, lo4.w, hi4.x, hi4.y, hi4.z, hi4.w};
            const int word0 = (pend_n0 >> 5) + wsel;
            const bool clear_pad = wsel == 0 && pend_n0 + kBN >= p.Ng;   // the last feature tile clears the row's padding words
            for (int i = tid / (2 * kBM); i < p.next_bits; i += PLANES_AT_ONCE) {
                uint32_t *dst = p.next_planes + (m * p.next_bits + i) * (int64_t)p.next_kw + word0;
                const uint32_t mask = 0x01010101u << i, mul = 0x10204080u >> i;
                uint32_t word = 0u;
#pragma unroll
                for (int g = 7; g >= 0; --g) word = __funnelshift_l((c4[g] & mask) * mul, word, 4);
                if (word0 < p.next_kw) *dst = word;
                if (clear_pad)
                    for (int wz = (pend_n0 >> 5) + 2; wz < p.next_kw; ++wz) dst[wz - word0] = 0u;
            }
        }
        pend_m0 = -1;
    };

    int tile = blockIdx.x;
    if (tile >= p.ntiles) return;
    TileSrc cur = prep_tile(tile);
    issue_stage(cur, 0, 0);
    int buf = 0;
    int code_buf = 0;                                  // code matrix that the next epilogue writes

    for (;;) {
        int acc[TM][4];
#pragma unroll
        for (int r = 0; r < TM; ++r)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[r][c] = 0;
        const int next_tile = tile + (int)gridDim.x;

        for (int stage = 0; stage < p.nstages; ++stage) {
            // the copies of this stage were issued one stage earlier; finish and re-code my own units
            cp_async_wait_all();
            recode_stage(stage, buf);
            __syncthreads();   // everybody's units are in place, and everybody is done reading buf^1
            if constexpr (FUSED) {
                if (pend_m0 >= 0) pack_pending();          // the previous tile's code matrix is complete as well
            }
            if (stage + 1 < p.nstages) {
                issue_stage(cur, stage + 1, buf ^ 1);
            } else if (next_tile < p.ntiles) {
                cur = prep_tile(next_tile);
                issue_stage(cur, 0, buf ^ 1);                                    // overlaps the epilogue too
            }

            const uint4 *a_s = smem + (size_t)buf * BUF_VEC;
            const uint4 *w_s = a_s + A_VEC;
            int nch = p.nfull - stage * kStageChunks;
            nch = nch > kStageChunks ? kStageChunks : nch;
            constexpr int GW = G9 ? 9 : 8;                                   // words per group
            const uint32_t *a_e = reinterpret_cast<const uint32_t *>(a_s + A_VEC + W_VEC);   // G9: ninth words
            const uint32_t *w_e = a_e + A_EXT;
#pragma unroll 1
            for (int ch = 0; ch < nch; ++ch) {
                uint32_t ta[TM][AB][GW];
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int i = 0; i < AB; ++i) {
#pragma unroll
                        for (int g = 0; g < 2; ++g) {
                            const uint4 v = a_s[((ch * 2 + g) * AB + i) * kBM + ty + 16 * r];
                            ta[r][i][4 * g + 0] = v.x; ta[r][i][4 * g + 1] = v.y;
                            ta[r][i][4 * g + 2] = v.z; ta[r][i][4 * g + 3] = v.w;
                        }
                        if constexpr (G9) ta[r][i][GW - 1] = a_e[(ch * AB + i) * kBM + ty + 16 * r];
                    }
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int j = 0; j < WB; ++j) {
                        uint32_t tw[GW];
#pragma unroll
                        for (int g = 0; g < 2; ++g) {
                            const uint4 v = w_s[((ch * 2 + g) * WB + j) * kBN + tx + 16 * c];
                            tw[4 * g + 0] = v.x; tw[4 * g + 1] = v.y; tw[4 * g + 2] = v.z; tw[4 * g + 3] = v.w;
                        }
                        if constexpr (G9) tw[GW - 1] = w_e[(ch * WB + j) * kBN + tx + 16 * c];
#pragma unroll
                        for (int r = 0; r < TM; ++r)
#pragma unroll
                            for (int i = 0; i < AB; ++i) {
                                if constexpr (G9) pair9(ta[r][i], tw, i + j, acc[r][c]);
                                else pair8(ta[r][i], tw, i + j, acc[r][c]);
                            }
                    }
            }
            if (!G9 && p.ntail > 0 && stage == p.nstages - 1) {
                const int ch = p.nfull % kStageChunks;
                // tail: up to 3 raw words, one popcount each (words past kwords are zero in both operands)
                uint32_t ta[TM][AB][3];
#pragma unroll
                for (int r = 0; r < TM; ++r)
#pragma unroll
                    for (int i = 0; i < AB; ++i) {
                        const uint4 v = a_s[((ch * 2) * AB + i) * kBM + ty + 16 * r];
                        ta[r][i][0] = v.x; ta[r][i][1] = v.y; ta[r][i][2] = v.z;
                    }
#pragma unroll
                for (int c = 0; c < 4; ++c)
#pragma unroll
                    for (int j = 0; j < WB; ++j) {
                        const uint4 v = w_s[((ch * 2) * WB + j) * kBN + tx + 16 * c];
#pragma unroll
                        for (int r = 0; r < TM; ++r)
#pragma unroll
                            for (int i = 0; i < AB; ++i) {
                                int cnt = __popc(ta[r][i][0] ^ v.x);
                                if (p.ntail > 1) cnt += __popc(ta[r][i][1] ^ v.y);
                                if (p.ntail > 2) cnt += __popc(ta[r][i][2] ^ v.z);
                                acc[r][c] += cnt * (1 << (i + j));
                            }
                    }
            }
            buf ^= 1;
        }

        // ---- epilogue: acc holds S = sum_ij 2^(i+j) X_ij.  out = n_valid*A*B - 2*S (Eq. 8), times alpha (Eq. 9).
        constexpr int AMAX = (1 << AB) - 1, PROD = AMAX * ((1 << WB) - 1);
        const int tile_n = FASTDIV ? (int)fastdiv((uint32_t)tile, p.tm_magic, p.tm_shift) : tile / p.tiles_m;
        const int64_t m0 = (int64_t)(tile - tile_n * p.tiles_m) * kBM;
        const int n0 = tile_n * kBN;
#pragma unroll
        for (int r = 0; r < TM; ++r) {
            const int64_t m = m0 + ty + 16 * r;
            const bool row_ok = m < p.Mg;
            if (!FUSED && !row_ok) continue;      // the fused encoder needs every lane at its ballots
            int n_valid = p.n_elems;
            int corr[4] = {0, 0, 0, 0};
            if (CONV && row_ok) {
                // Taps outside the image were staged as zero words: each contributed popc(w_j) to X_ij, i.e.
                // AMAX * tapsum[n][tap] to S, and must not be counted in the length.
                int wo, ho;
                if (FASTDIV && p.fast_pix) {
                    const uint32_t m32 = (uint32_t)m;
                    const uint32_t q = fastdiv(m32, p.wo_magic, p.wo_shift), img = fastdiv(m32, p.howo_magic, p.howo_shift);
                    wo = (int)(m32 - q * (uint32_t)p.Wo);
                    ho = (int)(q - img * (uint32_t)p.Ho);
                } else {
                    wo = (int)(m % p.Wo);
                    ho = (int)((m / p.Wo) % p.Ho);
                }
                const int hh = (GENERAL && p.transposed) ? ho + p.pad : ho * p.stride - p.pad;
                const int ww = (GENERAL && p.transposed) ? wo + p.pad : wo * p.stride - p.pad;
                int valid_taps = p.R * p.S;
                const bool interior = !GENERAL && hh >= 0 && ww >= 0 && hh + p.R <= p.H && ww + p.S <= p.W;
                if (!interior) {
                    valid_taps = 0;
                    for (int rr = 0; rr < p.R; ++rr)
                        for (int ss = 0; ss < p.S; ++ss) {
                            int hi = hh + rr, wi = ww + ss;
                            bool inside = hi >= 0 && hi < p.H && wi >= 0 && wi < p.W;
                            if (GENERAL) inside = tap_coord(p, hh, rr, p.H, hi) && tap_coord(p, ww, ss, p.W, wi);
                            if (inside) {
                                ++valid_taps;
                            } else {
#pragma unroll
                                for (int c = 0; c < 4; ++c) {
                                    const int n = n0 + tx + 16 * c;
                                    if (n < p.Ng) corr[c] += __ldg(p.tapsum + (int64_t)n * (p.R * p.S) + rr * p.S + ss);
                                }
                            }
                        }
                }
                n_valid = valid_taps * p.C;
            }
            float fv[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const int n = n0 + tx + 16 * c;
                if (!FUSED && n >= p.Ng) continue;
                const int32_t v = qnn_combine(n_valid * PROD, acc[r][c] - AMAX * corr[c]);
                fv[c] = __fmul_rn(__int2float_rn(v), p.alpha);
                if (FUSED && p.ch_gamma != nullptr && n < p.Ng)
                    fv[c] = __fmaf_rn(fv[c], __ldg(p.ch_gamma + n), p.ch_beta ? __ldg(p.ch_beta + n) : 0.0f);
                if (row_ok && n < p.Ng) {
                    if (p.acc) p.acc[m * p.Ng + n] = v;
                    if (p.out) p.out[m * p.ldo + n] = fv[c];
                }
            }
            if (FUSED && p.next_planes != nullptr) {
                // Next layer's encoder on the fp32 result (Alg. 1 forward: scale, then MBitEncoder), first half: the
                // codes of this thread's outputs go to the tile's code matrix in shared memory, one byte each
                // (0 outside the problem, so that padding bits come out as 0).
                uint8_t *codes = reinterpret_cast<uint8_t *>(smem + 2 * BUF_VEC) + code_buf * (kBM * kBN);   // [kBM][64]
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const int n = n0 + tx + 16 * c;
                    const uint32_t code = qnn_code_bits(fv[c], p.next_inv2s, p.next_half, p.next_lo, p.next_hi);
                    codes[(ty + 16 * r) * kBN + tx + 16 * c] = (row_ok && n < p.Ng) ? (uint8_t)code : (uint8_t)0;
                }
            }
        }
        if (FUSED && p.next_planes != nullptr) {
            pend_m0 = m0; pend_n0 = n0; pend_buf = code_buf;      // packed after the next barrier
            code_buf ^= 1;
        }
        tile = next_tile;
        if (tile >= p.ntiles) break;
    }
    if constexpr (FUSED) {
        if (pend_m0 >= 0) {                                // the last tile's codes
            __syncthreads();
            pack_pending();
        }
    }
}

// Peak probe: the inner loop of bgemm_tiled_kernel<2, 2> (same pair8, same register tile, same shared
// memory layout) running `iters` times over one resident stage: no global traffic, barriers or epilogue.
static __global__ void __launch_bounds__(kThreads, 2) probe_csa73_kernel(int iters, int32_t *sink) {
    constexpr int AB = 2, WB = 2, TM = 4, kBM = 64;
    constexpr int A_VEC = kStageChunks * 2 * AB * kBM, W_VEC = kStageChunks * 2 * WB * kBN;
    __shared__ uint4 sm[A_VEC + W_VEC];
    for (int i = threadIdx.x; i < A_VEC + W_VEC; i += kThreads) {
        const uint32_t h = (uint32_t)(i + 1) * 2654435761u + blockIdx.x * 40503u;
        sm[i] = make_uint4(h, h * 2246822519u, h ^ (h >> 7), h * 3266489917u + 1u);
    }
    __syncthreads();
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const uint4 *a_s = sm, *w_s = sm + A_VEC;
    int acc[TM][4];
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) acc[r][c] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll 1
        for (int ch = 0; ch < kStageChunks; ++ch) {
            uint32_t ta[TM][AB][8];
#pragma unroll
            for (int r = 0; r < TM; ++r)
#pragma unroll
                for (int i = 0; i < AB; ++i)
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const uint4 v = a_s[((ch * 2 + g) * AB + i) * kBM + ty + 16 * r];
                        ta[r][i][4 * g + 0] = v.x; ta[r][i][4 * g + 1] = v.y;
                        ta[r][i][4 * g + 2] = v.z; ta[r][i][4 * g + 3] = v.w;
                    }
#pragma unroll
            for (int c = 0; c < 4; ++c)
#pragma unroll
                for (int j = 0; j < WB; ++j) {
                    uint32_t tw[8];
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        const uint4 v = w_s[((ch * 2 + g) * WB + j) * kBN + tx + 16 * c];
                        tw[4 * g + 0] = v.x; tw[4 * g + 1] = v.y; tw[4 * g + 2] = v.z; tw[4 * g + 3] = v.w;
                    }
#pragma unroll
                    for (int r = 0; r < TM; ++r)
#pragma unroll
                        for (int i = 0; i < AB; ++i) pair8(ta[r][i], tw, i + j, acc[r][c]);
                }
        }
    }
    int s = 0;
#pragma unroll
    for (int r = 0; r < TM; ++r)
#pragma unroll
        for (int c = 0; c < 4; ++c) s += acc[r][c] * (r * 4 + c + 1);
    sink[blockIdx.x * kThreads + threadIdx.x] = s;
}
constexpr double kProbeCsa73WordsPerThreadIter = 8.0 * kStageChunks * 4 * 4 * 2 * 2;

template <int AB, int WB, int KIND, int TM, bool FUSED>
inline int launch_tiled_tmf(const Params &p, int sms, cudaStream_t st);

// The epilogue with the next layer's encoder is a separate instantiation for ab <= 4, so that the plain kernels
// carry none of its code; for ab >= 5 (16-row tiles, where the epilogue matters less) one instantiation serves both.
template <int AB, int WB, int KIND, int TM>
inline int launch_tiled_tm(const Params &p, int sms, cudaStream_t st) {
    constexpr int CONV = KIND;
    if constexpr (KIND == 2) {
        return launch_tiled_tmf<AB, WB, KIND, TM, false>(p, sms, st);      // no chaining epilogue for this kind
    } else if constexpr (AB >= 5) {
        return launch_tiled_tmf<AB, WB, CONV, TM, true>(p, sms, st);
    } else {
        if (p.next_planes != nullptr || p.ch_gamma != nullptr) return launch_tiled_tmf<AB, WB, CONV, TM, true>(p, sms, st);
        return launch_tiled_tmf<AB, WB, CONV, TM, false>(p, sms, st);
    }
}

template <int AB, int WB, int CONV, int TM, bool FUSED>
inline int launch_tiled_tmf(const Params &p, int sms, cudaStream_t st) {
    constexpr int kBM = 16 * TM;
    constexpr size_t ext = (CONV == 3) ? ((size_t)kStageChunks * (AB * kBM + WB * kBN) + 3u) / 4u * 16u : 0u;   // ninth words
    constexpr size_t smem = 2u * (kStageChunks * 2u * (AB * kBM + WB * kBN) * 16u + ext) + (FUSED ? 2u * (size_t)kBM * kBN : 0u);   // + the chaining epilogue's two code matrices
    if (smem > 48u * 1024u &&
        cudaFuncSetAttribute(bgemm_tiled_kernel<AB, WB, CONV, TM, FUSED>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem) != cudaSuccess)
        return QNN_E_CUDA;
    Params q = p;
    const int64_t tiles_m = (q.Mg + kBM - 1) / kBM, tiles_n = (q.Ng + kBN - 1) / kBN;
    if (tiles_m * tiles_n > 0x7fffffff) return QNN_E_RANGE;
    q.tiles_m = (int)tiles_m;
    q.ntiles = (int)(tiles_m * tiles_n);
    set_fastdiv((uint32_t)q.tiles_m, q.tm_magic, q.tm_shift);
    q.fast_pix = 0;
    if (CONV != 0 && q.Mg + kBM < (1ll << 31) && (int64_t)q.Ho * q.Wo < (1ll << 31) && q.Wo > 0 && q.Ho > 0) {
        set_fastdiv((uint32_t)q.Wo, q.wo_magic, q.wo_shift);
        set_fastdiv((uint32_t)((int64_t)q.Ho * q.Wo), q.howo_magic, q.howo_shift);
        q.fast_pix = 1;
    }
    if (CONV == 3) {               // one 9-word group per channel word, no tail
        q.nfull = q.cw;
        q.ntail = 0;
        q.nstages = (q.cw + kStageChunks - 1) / kStageChunks;
    } else {
        set_k_split(q);
    }
    // Short reductions: two persistent CTAs per SM walk the tiles and prefetch across tile boundaries, which
    // hides the first-stage latency that would otherwise dominate.  Long reductions: one CTA per tile measured
    // about 5% faster (the hardware's dynamic block placement balances better than the static walk).
    const bool persistent = q.nstages <= 3;
    const int per_sm = ((TM == 1 && AB == 4 && (CONV == 0 || CONV == 3)) || (AB == 1 && CONV != 2)) ? 3 : 2;
    const int grid = (persistent && q.ntiles > per_sm * sms) ? per_sm * sms : q.ntiles;
    bgemm_tiled_kernel<AB, WB, CONV, TM, FUSED><<<grid, kThreads, smem, st>>>(q);
    return cudaGetLastError() == cudaSuccess ? QNN_OK : QNN_E_CUDA;
}

// Share of the SMs' time spent on useful work when `tiles` equal tiles are handed out dynamically: an SM
// works through its tiles at the same rate whether one or two CTAs are resident, so the makespan is
// ceil(tiles / sms) tile-times.
inline double wave_efficiency(int64_t tiles, int64_t sms) {
    const int64_t rounds = (tiles + sms - 1) / sms;
    return (double)tiles / (double)(rounds * sms);
}

template <int AB, int WB, int CONV>
inline int launch_tiled(const Params &p, cudaStream_t st) {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return QNN_E_CUDA;
    if constexpr (AB <= 2) {
        // 64-row tiles reuse each weight word for four rows per thread; 32-row tiles measured ~5% slower per
        // operation but give twice as many tiles.  Take them only when that fills the SMs better (small problems).
        const int64_t tn = (p.Ng + kBN - 1) / kBN;
        const int64_t t64 = ((p.Mg + 63) / 64) * tn, t32 = ((p.Mg + 31) / 32) * tn;
        if constexpr (CONV != 2) {
            if (p.next_planes == nullptr && p.ch_gamma == nullptr && wave_efficiency(t32, sms) * 0.95 > wave_efficiency(t64, sms))
                return launch_tiled_tmf<AB, WB, CONV, 2, false>(p, sms, st);   // (no fused instantiation of this variant)
        }
        return launch_tiled_tm<AB, WB, CONV, 4>(p, sms, st);
    } else {
        // 4-bit activations: 16-row tiles (half the operand registers) and three CTAs per SM measured 3% faster than
        // 32-row tiles with two for the 3x3 convolutions with 9-word groups and 1.3-2% for fully-connected layers, but
        // 2.3% SLOWER for the 8-word convolution kernels; at 3 bits the same trade loses 5%
        if constexpr (AB == 4 && (CONV == 0 || CONV == 3)) return launch_tiled_tm<AB, WB, CONV, 1>(p, sms, st);
        return launch_tiled_tm<AB, WB, CONV, TileM<AB>::TM>(p, sms, st);
    }
}

// All weight widths for one activation width and operand kind; each (width, kind) is compiled in its own
// translation unit (tiled_ab<N>_fc.cu / _conv.cu / _gconv.cu) so that the kernel instantiations build in parallel.
template <int AB, int CONV>
inline int run_tiled_ab(int wb, const Params &p, cudaStream_t st) {
#define QNN_T(W_) \
    case W_: return launch_tiled<AB, W_, CONV>(p, st);
    switch (wb) {
        QNN_T(1) QNN_T(2) QNN_T(3) QNN_T(4) QNN_T(5) QNN_T(6) QNN_T(7) QNN_T(8)
        default: return QNN_E_ARG;
    }
#undef QNN_T
}
#define QNN_DECL(N_) \
    int run_tiled_ab##N_##_fc(int wb, const Params &p, cudaStream_t st); \
    int run_tiled_ab##N_##_conv(int wb, const Params &p, cudaStream_t st); \
    int run_tiled_ab##N_##_gconv(int wb, const Params &p, cudaStream_t st);
// 3x3 convolutions with 9-word groups (kind 3) exist for ab, wb <= 4
int run_tiled_conv3x3_ab1(int wb, const Params &p, cudaStream_t st);
int run_tiled_conv3x3_ab2(int wb, const Params &p, cudaStream_t st);
int run_tiled_conv3x3_ab3(int wb, const Params &p, cudaStream_t st);
int run_tiled_conv3x3_ab4(int wb, const Params &p, cudaStream_t st);
QNN_DECL(1) QNN_DECL(2) QNN_DECL(3) QNN_DECL(4) QNN_DECL(5) QNN_DECL(6) QNN_DECL(7) QNN_DECL(8)
#undef QNN_DECL

// kind: 0 = fully-connected, 1 = convolution, 2 = dilated / transposed convolution, 3 = 3x3 convolution (ab, wb <= 4)
inline int dispatch_tiled(int kind, int ab, int wb, const Params &p, cudaStream_t st) {
    if (kind == 3) {
        switch (ab) {
            case 1: return run_tiled_conv3x3_ab1(wb, p, st);
            case 2: return run_tiled_conv3x3_ab2(wb, p, st);
            case 3: return run_tiled_conv3x3_ab3(wb, p, st);
            case 4: return run_tiled_conv3x3_ab4(wb, p, st);
            default: return QNN_E_ARG;
        }
    }
#define QNN_CASE(N_) \
    case N_: return kind == 2 ? run_tiled_ab##N_##_gconv(wb, p, st) \
                  : kind == 1 ? run_tiled_ab##N_##_conv(wb, p, st) : run_tiled_ab##N_##_fc(wb, p, st);
    switch (ab) {
        QNN_CASE(1) QNN_CASE(2) QNN_CASE(3) QNN_CASE(4) QNN_CASE(5) QNN_CASE(6) QNN_CASE(7) QNN_CASE(8)
        default: return QNN_E_ARG;
    }
#undef QNN_CASE
}

}  // namespace qnn_tiled

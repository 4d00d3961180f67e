// qnn_encode_pack, qnn_pack_weights, qnn_absmax_f32: real tensors -> bit planes.
//
// Activations (qnn_encode_pack) take one of three kernels:
//  * encode_pack_lanes_kernel (source 16-byte aligned, ldx a multiple of 4: the usual case): a lane owns a
//    whole output word, i.e. 32 consecutive elements; see the comment above the kernel.
//  * encode_pack_kernel (any alignment): a warp owns 128 consecutive elements of one row, lane L reads
//    elements 32*j + L (four coalesced 128-byte requests) and one __ballot_sync per plane and j turns the
//    warp's 32 decisions into one canonical word (lane L -> bit L); lane i stores plane i's four words.
//  * encode_pack_tiny_kernel (rows of at most 8 elements, or at most 32 from an unaligned source): a thread owns a row.
// The weight packer (offline) uses the ballot scheme as well.
#include "qnn_internal.cuh"
#include <string.h>

namespace {

constexpr int kEncThreads = 256;

// The encoders here take the code from qnn_code_bits (no float->int conversion: those run on the XU pipe, whose
// rate made them the bottleneck of this kernel -- ncu showed XU saturated and DRAM at half its rate).
constexpr uint32_t kEncMagicBits = 0x4B000000u;             // bit pattern of 2^23, the offset in qnn_code_bits
__device__ __forceinline__ uint32_t enc_code_bits(float x, float inv2s, float half, float lo, float hi) {
    return qnn_code_bits(x, inv2s, half, lo, hi);
}
__device__ __forceinline__ int enc_code_t(float x, float inv2s, float half, float lo, float hi) {
    return (int)(qnn_code_bits(x, inv2s, half, lo, hi) & 0xffu);
}

// One- and two-bit codes are decided by comparisons alone.  The quantizer is a non-decreasing step function of x,
// so t = [x >= t_lo] + [x > 0] + [x >= t_hi] for two bits (the middle step, between codes -1 and +1, is at 0 with
// 0 itself on the lower side) and t = [x > 0] for one bit; t_lo / t_hi are the smallest floats at which the
// quantizer's own formula (fused multiply-add, then floor / ceil - 1) reaches the next code, found on the host
// with the same binary32 arithmetic.  NaN fails every comparison (t = 0, the most negative code); with a fused
// ReLU every x <= 0 and NaN take the code of 0, i.e. the lowest step counts as passed.
struct EncThresholds { float t_lo, t_hi; };

template <int BITS, bool RELU>
__device__ __forceinline__ void enc_ballots_small(float x, const EncThresholds th, uint32_t (&b)[BITS]) {
    const bool c_mid = x > 0.0f;
    if (BITS == 1) {
        b[0] = __ballot_sync(0xffffffffu, c_mid);
    } else {
        const bool c_hi = x >= th.t_hi;
        const bool c_lo = RELU ? true : (x >= th.t_lo);
        b[BITS - 1] = __ballot_sync(0xffffffffu, c_mid);                   // t >= 2 exactly when x > 0
        b[0] = __ballot_sync(0xffffffffu, (c_lo != c_mid) != c_hi);        // parity of the steps passed
    }
}

// A unit is 128 consecutive elements: four ballots per plane give four canonical words.  For rows
// longer than 64 elements a unit is a 128-element segment of one row (RPU = 1); for shorter rows
// (33..64 elements, from an unaligned source) a unit spans RPU = 2 whole rows so
// that the lanes stay busy.  UN units are loaded before the first ballot, so 4*UN independent
// 128-byte requests per warp are in flight.  Unit indices advance incrementally (no division in the loop).
// MODE 0: any width, codes from the quantizer's formula; MODE 1 / 2 (BITS <= 2, RPU = 1, no rowsum): codes from
// comparisons against precomputed thresholds, without / with the fused ReLU.
template <int BITS, int UN, int RPU, bool FULL, int MODE>
__global__ void __launch_bounds__(kEncThreads)
encode_pack_kernel(const float *__restrict__ x, int64_t rows, int k, int64_t ldx, float inv2s, float lo, float hi,
                   const EncThresholds th, uint32_t *__restrict__ planes, int32_t *__restrict__ rowsum,
                   int groups_per_row, int segs_per_row, int kw, int64_t first_row_step, int first_grp_step) {
    static_assert(MODE == 0 || (BITS <= 2 && RPU == 1), "threshold mode");
    const float half = (float)(1 << (BITS - 1));
    constexpr int SPAN = 128 / RPU;                       // elements of one row inside a unit (RPU > 1)
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kEncThreads + threadIdx.x) >> 5;
    // group g = (row-unit, group of UN segments); RPU > 1 has one group per row-unit
    int64_t ru = warp0 / groups_per_row;                  // row (RPU = 1) or index of a bundle of RPU rows
    int grp = (int)(warp0 - ru * groups_per_row);
    const int64_t n_ru = (RPU == 1) ? rows : ((rows + RPU - 1) / RPU + UN - 1) / UN;
    for (; ru < n_ru;) {
        float v[UN][4];
#pragma unroll
        for (int q = 0; q < UN; ++q) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                int64_t row;
                int kk;
                if (RPU == 1) {
                    row = ru;
                    kk = (grp * UN + q) * 128 + 32 * j + lane;
                } else {
                    row = (ru * UN + q) * RPU + (32 * j) / SPAN;
                    kk = (32 * j) % SPAN + lane;
                }
                const bool live = (RPU == 1) ? ((grp * UN + q) < segs_per_row) : (row < rows);
                v[q][j] = (live && (FULL || kk < k)) ? __ldcs(x + row * ldx + kk) : 0.0f;
            }
        }
#pragma unroll
        for (int q = 0; q < UN; ++q) {
            const int seg = grp * UN + q;
            if (RPU == 1 && seg >= segs_per_row) break;                            // warp-uniform
            int t[4];
            uint32_t b[BITS][4];
            if constexpr (MODE != 0) {
                // (rows that end inside the unit were loaded as 0.0f; their padding bits are cleared below)
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    uint32_t bj[BITS];
                    enc_ballots_small<BITS, MODE == 2>(v[q][j], th, bj);
                    const int k0 = seg * 128 + 32 * j;                          // warp-uniform
                    const uint32_t keep = FULL ? 0xffffffffu : (k0 + 32 <= k ? 0xffffffffu : (k0 >= k ? 0u : (0xffffffffu >> (32 - (k - k0)))));
#pragma unroll
                    for (int i = 0; i < BITS; ++i) b[i][j] = bj[i] & keep;
                    t[j] = 0;
                }
            } else {
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int kk = (RPU == 1) ? seg * 128 + 32 * j + lane : (32 * j) % SPAN + lane;
                    const int code = enc_code_t(v[q][j], inv2s, half, lo, hi);
                    t[j] = (FULL || kk < k) ? code : 0;                                // padding bits are 0
                }
#pragma unroll
                for (int i = 0; i < BITS; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) b[i][j] = __ballot_sync(0xffffffffu, t[j] & (1 << i));
            }
            if (RPU == 1) {
                // lane i stores plane i (each lane's address already points at its own plane): one predicated
                // 16-byte store per plane instead of moving the ballots into the storing lanes' registers
                uint32_t *dst = planes + (ru * BITS + (lane < BITS ? lane : 0)) * (int64_t)kw + seg * 4;
#pragma unroll
                for (int i = 0; i < BITS; ++i)
                    if (lane == i) *reinterpret_cast<uint4 *>(dst) = make_uint4(b[i][0], b[i][1], b[i][2], b[i][3]);
                if (rowsum != nullptr) {
                    int s = t[0] + t[1] + t[2] + t[3];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                    if (lane == 0) atomicAdd(rowsum + ru, s);
                }
            } else {
                // lane r*BITS + i stores plane i of bundle row r: words [b(r-th span)...], rest 0 (kw == 4)
                constexpr int WPR = SPAN / 32;            // ballots per row: 2 or 1
                uint4 mine = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int r = 0; r < RPU; ++r)
#pragma unroll
                    for (int i = 0; i < BITS; ++i)
                        if (lane == r * BITS + i)
                            mine = make_uint4(b[i][r * WPR], WPR == 2 ? b[i][r * WPR + 1] : 0u, 0u, 0u);
                const int64_t row = (ru * UN + q) * RPU + lane / BITS;
                if (lane < RPU * BITS && row < rows)
                    *reinterpret_cast<uint4 *>(planes + (row * BITS + lane % BITS) * (int64_t)kw) = mine;
                if (rowsum != nullptr) {
#pragma unroll
                    for (int r = 0; r < RPU; ++r) {
                        int s = 0;
#pragma unroll
                        for (int jj = 0; jj < WPR; ++jj) s += t[r * WPR + jj];
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
                        const int64_t rr = (ru * UN + q) * RPU + r;
                        if (lane == 0 && rr < rows) rowsum[rr] = s;
                    }
                }
            }
        }
        // advance by the number of warps in the grid without dividing
        grp += first_grp_step;
        ru += first_row_step;
        if (grp >= groups_per_row) { grp -= groups_per_row; ++ru; }
    }
}


// ---- per-lane packing kernel (the default whenever x is 16-byte aligned and ldx is a multiple of 4) ----------------
// A warp-wide ballot costs about four ALU-pipe slots per lane on this GPU, so turning 32 lanes' decisions into a
// word that way makes the encoder ALU-bound at 3 or more bits.  Here a lane owns one whole output word instead: 32
// consecutive elements of a row.  A warp takes a unit of 32 words (4 KB of floats): every lane loads eight coalesced
// float4 (all eight in flight before the first is used), quantizes each to four codes packed into the bytes of one
// register, and hands that register through a small per-warp slice of shared memory to the lane that owns the word;
// the owner reads its eight registers of codes back (two 16-byte reads) and moves bit i of each byte into a nibble
// with one mask and one multiply:
//   ((c & (0x01010101 << i)) * (0x10204080 >> i)) >> 28 = b3 b2 b1 b0   (partial products land on distinct bits)
// which a funnel shift appends to plane i's word: 2 ALU operations + 1 multiply per 4 elements and plane.
// (Copying the floats themselves to shared memory with cp.async was tried first: 16-byte cp.async retires about
// one lane per clock per SM here, which capped the kernel at 4.2 TB/s.)
// A unit is R rows x S words with R*S = 32 and S a power of two covering min(kw, 32) words, so that short rows (NHWC
// activations with few channels) keep all lanes busy.  Plane words of one row segment are stored by consecutive
// lanes (coalesced).  Padding words and the bits past k are written as 0.
// Shared-memory slot of word `item` of the unit: 8 registers + 4 words of padding after every fourth item, which
// makes both the 4-byte writes (lane -> item lane/8 + 4j, register lane%8) and the 16-byte reads conflict-free.
__device__ __forceinline__ int enc_slot(int item) { return 8 * item + 4 * (item >> 2); }
constexpr int kLaneSlotWords = 8 * 32 + 4 * 8;

template <int BITS, int LOG2S>
__global__ void __launch_bounds__(kEncThreads, 4)
encode_pack_lanes_kernel(const float *__restrict__ x, int64_t rows, int k, int64_t ldx, float inv2s, float lo, float hi,
                         uint32_t *__restrict__ planes, int32_t *__restrict__ rowsum, int kw, int segs, int64_t n_units) {
    __shared__ __align__(16) uint32_t enc_codes[kEncThreads / 32][kLaneSlotWords];
    const float half = (float)(1 << (BITS - 1));
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t *sc = enc_codes[warp];
    constexpr int S = 1 << LOG2S, R = 32 >> LOG2S;
    const int64_t nwarps = (int64_t)gridDim.x * (kEncThreads / 32);
    const int ca = lane >> 3, cc = lane & 7;                 // load role: word ca + 4j of the unit, 16-byte piece cc
    // Piece j of this lane is word ca + 4j of the unit.  S >= 4: row j / (S/4) of the unit, and within that row's
    // segment element 128*(j % (S/4)) + 4*lane.  S < 4 (rows of at most 64 elements): row (ca >> LOG2S) + (4/S)*j,
    // element 32*(ca % S) + 4*cc.  With S fixed at compile time every piece is a constant offset from one base.
    constexpr int JPR = S >= 4 ? S / 4 : 1;                  // pieces per lane and row (S >= 4)
    constexpr int RSTEP = S >= 4 ? 0 : 4 / S;                // rows between consecutive pieces of a lane (S < 4)
    const int row0 = S >= 4 ? 0 : (ca >> LOG2S);             // row of piece 0 within the unit
    const int el0 = S >= 4 ? 4 * lane : 32 * (ca & (S - 1)) + 4 * cc;   // element of piece 0 within the segment

    for (int64_t u = (int64_t)blockIdx.x * (kEncThreads / 32) + warp; u < n_units; u += nwarps) {
        const int64_t rg = u / segs;                         // warp-uniform
        const int seg = (int)(u - rg * segs);
        const float *xl = x + (rg * R + row0) * ldx + (int64_t)seg * S * 32 + el0;
        const int64_t rows_left = rows - rg * R;
        const int k_left = k - seg * S * 32;                 // elements of the row from this segment on (may be <= 0)
        float4 f[8];
        if (rows_left >= R && k_left >= S * 32) {            // the whole unit is inside the tensor
#pragma unroll
            for (int j = 0; j < 8; ++j)
                f[j] = __ldcs(reinterpret_cast<const float4 *>(xl + (int64_t)(S >= 4 ? j / JPR : RSTEP * j) * ldx +
                                                               (S >= 4 ? 128 * (j % JPR) : 0)));
        } else {
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int dr = S >= 4 ? j / JPR : RSTEP * j, de = S >= 4 ? 128 * (j % JPR) : 0;
                const int r = row0 + dr, e = el0 + de;
                const float *src = xl + (int64_t)dr * ldx + de;
                f[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                if (r < rows_left) {
                    if (e + 4 <= k_left) {
                        f[j] = __ldcs(reinterpret_cast<const float4 *>(src));
                    } else if (e < k_left) {                 // the row ends inside this piece
                        f[j].x = src[0];
                        if (e + 1 < k_left) f[j].y = src[1];
                        if (e + 2 < k_left) f[j].z = src[2];
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            // four codes in the bytes of one register; each operand is 2^23's pattern + t, the shifted ones lose
            // that pattern's bits off the top, the unshifted one's is subtracted
            const uint32_t t0 = enc_code_bits(f[j].x, inv2s, half, lo, hi), t1 = enc_code_bits(f[j].y, inv2s, half, lo, hi);
            const uint32_t t2 = enc_code_bits(f[j].z, inv2s, half, lo, hi), t3 = enc_code_bits(f[j].w, inv2s, half, lo, hi);
            sc[enc_slot(ca + 4 * j) + cc] = t0 + (t1 << 8) + (t2 << 16) + (t3 << 24) - kEncMagicBits;
        }
        __syncwarp();
        const uint4 c_lo = *reinterpret_cast<const uint4 *>(sc + enc_slot(lane));
        const uint4 c_hi = *reinterpret_cast<const uint4 *>(sc + enc_slot(lane) + 4);
        __syncwarp();                                        // all reads done before the next unit's writes
        const uint32_t c4[8] = {c_lo.x, c_lo.y, c_lo.z, c_lo.w, c_hi.x, c_hi.y, c_hi.z, c_hi.w};
        uint32_t word[BITS];
#pragma unroll
        for (int i = 0; i < BITS; ++i) word[i] = 0u;
#pragma unroll
        for (int g = 7; g >= 0; --g) {                       // last group first: each append shifts the word left
#pragma unroll
            for (int i = 0; i < BITS; ++i) {
                const uint32_t prod = (c4[g] & (0x01010101u << i)) * (0x10204080u >> i);
                word[i] = __funnelshift_l(prod, word[i], 4);
            }
        }
        const int64_t row = rg * R + (lane >> LOG2S);
        const int w = seg * S + (lane & (S - 1));
        if (row < rows && w < kw) {
            const int len = k - 32 * w;
            const uint32_t mask = len >= 32 ? 0xffffffffu : (len <= 0 ? 0u : ((1u << len) - 1u));
            uint32_t *dst = planes + (row * BITS) * (int64_t)kw + w;
#pragma unroll
            for (int i = 0; i < BITS; ++i) dst[(int64_t)i * kw] = word[i] & mask;
            if constexpr (S < 4) {
                // rows of one or two words: the row's storage is four words, the lane of word 0 clears the rest
                if (w == 0) {
#pragma unroll
                    for (int i = 0; i < BITS; ++i) {
                        if (S == 1) dst[(int64_t)i * kw + 1] = 0u;
                        *reinterpret_cast<uint2 *>(dst + (int64_t)i * kw + 2) = make_uint2(0u, 0u);
                    }
                }
            }
            if (rowsum != nullptr && len > 0) {
                int sum = 0;
#pragma unroll
                for (int i = 0; i < BITS; ++i) sum += __popc(word[i] & mask) << i;
                atomicAdd(rowsum + row, sum);
            }
        }
    }
}

// Rows of a few elements (a first layer's 3-channel pixels): one thread per row.  The thread reads its k <= 32 values,
// builds the row's single word of every plane itself and stores it with the three padding words as one 16-byte
// vector; consecutive threads hold consecutive rows, so a warp's stores fill whole lines.  Works for any alignment
// of x and any ldx.  The work per element grows with bits (three logic operations per element and plane), which is
// why longer rows take the kernels above; here the stores (16 bytes per row and plane) dominate.
template <int BITS>
__global__ void __launch_bounds__(kEncThreads)
encode_pack_tiny_kernel(const float *__restrict__ x, int64_t rows, int k, int64_t ldx, float inv2s, float lo, float hi,
                        uint32_t *__restrict__ planes, int32_t *__restrict__ rowsum) {
    const float half = (float)(1 << (BITS - 1));
    for (int64_t row = (int64_t)blockIdx.x * kEncThreads + threadIdx.x; row < rows; row += (int64_t)gridDim.x * kEncThreads) {
        const float *src = x + row * ldx;
        uint32_t word[BITS];
#pragma unroll
        for (int i = 0; i < BITS; ++i) word[i] = 0u;
        int sum = 0;
        for (int c = 0; c < k; ++c) {
            const uint32_t t = qnn_code_bits(__ldg(src + c), inv2s, half, lo, hi) & 0xffu;
            sum += (int)t;
#pragma unroll
            for (int i = 0; i < BITS; ++i) word[i] |= ((t >> i) & 1u) << c;
        }
        uint4 *dst = reinterpret_cast<uint4 *>(planes + row * BITS * 4);
#pragma unroll
        for (int i = 0; i < BITS; ++i) dst[i] = make_uint4(word[i], 0u, 0u, 0u);
        if (rowsum != nullptr) rowsum[row] = sum;
    }
}

// Offline weight packer: one warp per (output feature, group of 4 words).  A word
// covers 32 input channels of one tap; the source index follows the layout flag.
template <int BITS>
__global__ void __launch_bounds__(kEncThreads)
pack_weights_kernel(const float *__restrict__ w, int n_out, int taps, int c_in, int layout, float inv2s, float lo,
                    float hi, uint32_t *__restrict__ planes, int kw, int cw) {
    const float half = (float)(1 << (BITS - 1));
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kEncThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kEncThreads) >> 5;
    const int groups = kw / 4;
    const int64_t units = (int64_t)n_out * groups;
    for (int64_t u = warp0; u < units; u += nwarps) {
        const int n = (int)(u / groups);
        const int g = (int)(u - (int64_t)n * groups);
        int t[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int word = g * 4 + j;
            const int tap = word / cw;
            const int c = (word - tap * cw) * 32 + lane;
            t[j] = 0;
            if (tap < taps && c < c_in) {
                int64_t idx;
                if (layout == QNN_W_NTC) idx = ((int64_t)n * taps + tap) * c_in + c;
                else if (layout == QNN_W_TCN) idx = ((int64_t)tap * c_in + c) * n_out + n;
                else idx = ((int64_t)n * c_in + c) * taps + tap;
                t[j] = qnn_code_t(w[idx], inv2s, half, lo, hi);
            }
        }
        uint4 mine = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
        for (int i = 0; i < BITS; ++i) {
            uint32_t b0 = __ballot_sync(0xffffffffu, (t[0] >> i) & 1);
            uint32_t b1 = __ballot_sync(0xffffffffu, (t[1] >> i) & 1);
            uint32_t b2 = __ballot_sync(0xffffffffu, (t[2] >> i) & 1);
            uint32_t b3 = __ballot_sync(0xffffffffu, (t[3] >> i) & 1);
            if (lane == i) mine = make_uint4(b0, b1, b2, b3);
        }
        if (lane < BITS)
            *reinterpret_cast<uint4 *>(planes + ((int64_t)n * BITS + lane) * kw + g * 4) = mine;
    }
}

// tapsum[n][tap] = sum_c t(n, tap, c), read back from the packed planes (bit i of t has weight 2^i).
__global__ void __launch_bounds__(kEncThreads)
weights_tapsum_kernel(const uint32_t *__restrict__ planes, int n_out, int taps, int bits, int kw, int cw,
                      int32_t *__restrict__ tapsum) {
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kEncThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kEncThreads) >> 5;
    const int64_t units = (int64_t)n_out * taps;
    for (int64_t u = warp0; u < units; u += nwarps) {
        const int n = (int)(u / taps);
        const int tap = (int)(u - (int64_t)n * taps);
        int s = 0;
        for (int i = 0; i < bits; ++i) {
            const uint32_t *p = planes + ((int64_t)n * bits + i) * kw + (int64_t)tap * cw;
            for (int c = lane; c < cw; c += 32) s += __popc(p[c]) << i;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) tapsum[u] = s;
    }
}

__global__ void __launch_bounds__(256) absmax_kernel(const float *__restrict__ x, size_t n, unsigned *out) {
    float m = 0.0f;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        m = fmaxf(m, fabsf(x[i]));                       // fmaxf drops NaN operands
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    // non-negative floats order like their bit patterns
    if ((threadIdx.x & 31) == 0) atomicMax(out, __float_as_uint(m));
}

int grid_for(int64_t warps_needed) {
    int64_t blocks = qnn_ceil_div(warps_needed, kEncThreads / 32);
    const int64_t cap = 148 * 8 * 4;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    return (int)blocks;
}

// Order-preserving map between floats and unsigned keys (negative floats reversed below the positive ones).
inline uint32_t enc_key_of(float f) {
    uint32_t u;
    memcpy(&u, &f, 4);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
inline float enc_float_of(uint32_t key) {
    const uint32_t u = (key & 0x80000000u) ? (key & 0x7fffffffu) : ~key;
    float f;
    memcpy(&f, &u, 4);
    return f;
}
// Smallest finite float x with pred(fmaf(x, inv2s, 2.0f)) true, for a predicate that is monotone in x
// (false below, true above), searched by bisection over the float ordering.
template <typename Pred>
inline float enc_first_true(float inv2s, Pred pred) {
    uint32_t lo = enc_key_of(-3.0e38f), hi = enc_key_of(3.0e38f);      // pred(lo) false, pred(hi) true
    while (hi - lo > 1u) {
        const uint32_t mid = lo + (hi - lo) / 2u;
        if (pred(fmaf(enc_float_of(mid), inv2s, 2.0f))) hi = mid; else lo = mid;
    }
    return enc_float_of(hi);
}
// Two-bit thresholds (see EncThresholds): t reaches 1 where ceil(v) - 1 >= 1, i.e. v > 1, and 3 where floor(v) >= 3.
inline EncThresholds enc_thresholds2(float inv2s) {
    EncThresholds th;
    th.t_lo = enc_first_true(inv2s, [](float v) { return v > 1.0f; });
    th.t_hi = enc_first_true(inv2s, [](float v) { return v >= 3.0f; });
    return th;
}

template <int BITS>
void launch_encode(const float *x, int64_t rows, int k, int64_t ldx, float scale, bool relu, uint32_t *planes,
                   int32_t *rowsum, cudaStream_t st) {
    constexpr int UN = 4;
    const float inv2s = 1.0f / (2.0f * scale);
    float lo, hi;
    qnn_clamp_bounds(BITS, scale, relu, &lo, &hi);
    const int kw = (int)qnn_row_words_i(k);
    const bool lanes_ok = qnn_aligned(x, 16) && ldx % 4 == 0;
    if (k <= 8 || (k <= 32 && !lanes_ok)) {
        // one thread per row (kw == 4: one real word and three padding words per plane)
        int64_t blocks = qnn_ceil_div(rows, kEncThreads);
        if (blocks > 148 * 16) blocks = 148 * 16;
        encode_pack_tiny_kernel<BITS><<<(int)blocks, kEncThreads, 0, st>>>(x, rows, k, ldx, inv2s, lo, hi, planes, rowsum);
        return;
    }
    if (lanes_ok) {
        // per-lane packing kernel; the ballot kernels below remain for unaligned inputs
        // S = 2^log2s words per row segment: the real words of the row when they are at most 32 (rows of one or two
        // words get S = 1 or 2; their padding words are cleared by the lane of word 0), else 32 with several segments
        const int cw_real = (k + 31) / 32;
        int log2s = 0;
        while ((1 << log2s) < cw_real && log2s < 5) ++log2s;
        const int segs_l = log2s < 2 ? 1 : (kw + (1 << log2s) - 1) >> log2s;
        const int rpu_l = 32 >> log2s;
        const int64_t n_units = qnn_ceil_div(rows, rpu_l) * segs_l;
        int dev = 0, sms = 148;
        if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        int64_t blocks = qnn_ceil_div(n_units, kEncThreads / 32);
        if (blocks > 4 * (int64_t)sms) blocks = 4 * (int64_t)sms;
#define QNN_ENC_LANES(L_) \
    encode_pack_lanes_kernel<BITS, L_><<<(int)blocks, kEncThreads, 0, st>>>(x, rows, k, ldx, inv2s, lo, hi, planes, rowsum, kw, segs_l, n_units)
        switch (log2s) {
            case 0: QNN_ENC_LANES(0); break;
            case 1: QNN_ENC_LANES(1); break;
            case 2: QNN_ENC_LANES(2); break;
            case 3: QNN_ENC_LANES(3); break;
            case 4: QNN_ENC_LANES(4); break;
            default: QNN_ENC_LANES(5); break;
        }
#undef QNN_ENC_LANES
        return;
    }
    const int segs = kw / 4;
    int groups;
    int64_t total;                                   // warp-level work items
    const int rpu = (k <= 64) ? 2 : 1;               // (rows of at most 32 elements never get here: one thread per row above)
    if (rpu == 1) {
        groups = (int)qnn_ceil_div(segs, UN);
        total = rows * groups;
    } else {
        groups = 1;
        total = qnn_ceil_div(qnn_ceil_div(rows, rpu), UN);
    }
    const int grid = grid_for(total);
    const int64_t nwarps = (int64_t)grid * (kEncThreads / 32);
    const int64_t row_step = nwarps / groups;
    const int grp_step = (int)(nwarps % groups);
    EncThresholds th = {0.0f, 0.0f};
#define QNN_ENC(RPU_, FULL_, MODE_)                                                                  \
    encode_pack_kernel<BITS, UN, RPU_, FULL_, MODE_><<<grid, kEncThreads, 0, st>>>(                  \
        x, rows, k, ldx, inv2s, lo, hi, th, planes, rowsum, groups, segs, kw, row_step, grp_step)
    if (rpu == 1) {
        if constexpr (BITS <= 2) {
            if (rowsum == nullptr) {
                if (BITS == 2) th = enc_thresholds2(inv2s);
                if (relu) { if (k % 128 == 0) QNN_ENC(1, true, 2); else QNN_ENC(1, false, 2); }
                else      { if (k % 128 == 0) QNN_ENC(1, true, 1); else QNN_ENC(1, false, 1); }
                return;
            }
        }
        if (k % 128 == 0) QNN_ENC(1, true, 0); else QNN_ENC(1, false, 0);
    } else {
        if (k == 64) QNN_ENC(2, true, 0); else QNN_ENC(2, false, 0);
    }
#undef QNN_ENC
}

template <int BITS>
void launch_pack_w(const float *w, int n_out, int taps, int c_in, int layout, float scale, uint32_t *planes,
                   cudaStream_t st) {
    const int kw = (int)qnn_w_row_words_i(taps, c_in);
    const int cw = (c_in + 31) / 32;
    const float inv2s = 1.0f / (2.0f * scale);
    float lo, hi;
    qnn_clamp_bounds(BITS, scale, false, &lo, &hi);
    pack_weights_kernel<BITS><<<grid_for((int64_t)n_out * (kw / 4)), kEncThreads, 0, st>>>(w, n_out, taps, c_in, layout,
                                                                                      inv2s, lo, hi, planes, kw, cw);
}

}  // namespace

#define QNN_DISPATCH_BITS(bits, CALL)          \
    switch (bits) {                            \
        case 1: CALL(1); break;                \
        case 2: CALL(2); break;                \
        case 3: CALL(3); break;                \
        case 4: CALL(4); break;                \
        case 5: CALL(5); break;                \
        case 6: CALL(6); break;                \
        case 7: CALL(7); break;                \
        default: CALL(8); break;               \
    }

int qnn_check_encode_pack(const float *x, int64_t rows, int k, int64_t ldx, int bits, float scale, unsigned flags,
                          const uint32_t *planes, const int32_t *rowsum) {
    if (!x || !planes || rows <= 0 || k <= 0 || ldx < k || !qnn_bits_ok(bits) || (flags & ~QNN_RELU)) return QNN_E_ARG;
    if (!(scale >= 1e-30f) || !(scale <= 1e30f)) return QNN_E_SCALE;   // also rejects NaN, 0, negatives, infinities
    if (!qnn_aligned(planes, 16) || !qnn_aligned(x, 4) || (rowsum && !qnn_aligned(rowsum, 4))) return QNN_E_ALIGN;
    if (k > (1 << 30) || rows > ((int64_t)1 << 40)) return QNN_E_RANGE;
    return QNN_OK;
}

extern "C" int qnn_encode_pack(const float *x, int64_t rows, int k, int64_t ldx, int bits, float scale,
                               unsigned flags, uint32_t *planes, int32_t *rowsum, void *stream) {
    if (const int rc = qnn_check_encode_pack(x, rows, k, ldx, bits, scale, flags, planes, rowsum)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool relu = (flags & QNN_RELU) != 0;
    if (rowsum && (k > 64 || (qnn_aligned(x, 16) && ldx % 4 == 0)) && cudaMemsetAsync(rowsum, 0, (size_t)rows * sizeof(int32_t), st) != cudaSuccess)
        return QNN_E_CUDA;
#define CALL(B) launch_encode<B>(x, rows, k, ldx, scale, relu, planes, rowsum, st)
    QNN_DISPATCH_BITS(bits, CALL)
#undef CALL
    return qnn_launch_status();
}

extern "C" int qnn_pack_weights(const float *w, int n_out, int taps, int c_in, int layout, int bits, float scale,
                                void *packed, void *stream) {
    if (!w || !packed || n_out <= 0 || taps <= 0 || c_in <= 0 || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (layout != QNN_W_NTC && layout != QNN_W_TCN && layout != QNN_W_NCT) return QNN_E_ARG;
    if (!(scale >= 1e-30f) || !(scale <= 1e30f)) return QNN_E_SCALE;   // also rejects NaN, 0, negatives, infinities
    if (!qnn_aligned(packed, 16) || !qnn_aligned(w, 4)) return QNN_E_ALIGN;
    const int64_t kw = qnn_w_row_words_i(taps, c_in);
    if (kw > (1 << 26) || (int64_t)n_out * bits * kw > ((int64_t)1 << 40)) return QNN_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t *planes = static_cast<uint32_t *>(packed);
    int32_t *tapsum = reinterpret_cast<int32_t *>(planes + (int64_t)n_out * bits * kw);
#define CALL(B) launch_pack_w<B>(w, n_out, taps, c_in, layout, scale, planes, st)
    QNN_DISPATCH_BITS(bits, CALL)
#undef CALL
    if (cudaGetLastError() != cudaSuccess) return QNN_E_CUDA;
    const int cw = (c_in + 31) / 32;
    weights_tapsum_kernel<<<grid_for((int64_t)n_out * taps), kEncThreads, 0, st>>>(planes, n_out, taps, bits, (int)kw,
                                                                                cw, tapsum);
    return qnn_launch_status();
}

extern "C" int qnn_absmax_f32(const float *x, size_t n, float *out, void *stream) {
    if (!x || !out || n == 0) return QNN_E_ARG;
    if (!qnn_aligned(x, 4) || !qnn_aligned(out, 4)) return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemsetAsync(out, 0, sizeof(float), st) != cudaSuccess) return QNN_E_CUDA;
    size_t blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    absmax_kernel<<<(int)blocks, 256, 0, st>>>(x, n, reinterpret_cast<unsigned *>(out));
    return qnn_launch_status();
}

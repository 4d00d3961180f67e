// qnn_encode_pack, qnn_pack_weights, qnn_absmax_f32: real tensors -> bit planes.
//
// Both packers are bandwidth-bound streaming kernels.  A warp owns 128 consecutive
// elements of one row: lane L reads elements 32*j + L (j = 0..3, four coalesced
// 128-byte requests), quantizes them, and one __ballot_sync per plane and j turns
// the warp's 32 decisions into one canonical word (lane L -> bit L).  Lane i then
// holds the four words of plane i and stores them as one 16-byte vector.
#include "qnn_internal.cuh"

namespace {

constexpr int kEncThreads = 256;

// A unit is 128 consecutive elements: four ballots per plane give four canonical words.  For rows
// longer than 64 elements a unit is a 128-element segment of one row (RPU = 1); for shorter rows
// (NHWC activations with few channels) a unit spans RPU = 2 (k <= 64) or 4 (k <= 32) whole rows so
// that the lanes stay busy.  UN units are loaded before the first ballot, so 4*UN independent
// 128-byte requests per warp are in flight.  Unit indices advance incrementally (no division in the loop).
template <int BITS, int UN, int RPU, bool FULL>
__global__ void __launch_bounds__(kEncThreads)
encode_pack_kernel(const float *__restrict__ x, int64_t rows, int k, int64_t ldx, float inv2s, float lo, float hi,
                   uint32_t *__restrict__ planes, int32_t *__restrict__ rowsum, int groups_per_row, int segs_per_row,
                   int kw, int64_t first_row_step, int first_grp_step) {
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
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const int kk = (RPU == 1) ? seg * 128 + 32 * j + lane : (32 * j) % SPAN + lane;
                const int code = qnn_code_t(v[q][j], inv2s, half, lo, hi);
                t[j] = (FULL || kk < k) ? code : 0;                                // padding bits are 0
            }
            uint32_t b[BITS][4];
#pragma unroll
            for (int i = 0; i < BITS; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) b[i][j] = __ballot_sync(0xffffffffu, t[j] & (1 << i));
            if (RPU == 1) {
                uint4 mine = make_uint4(b[0][0], b[0][1], b[0][2], b[0][3]);
#pragma unroll
                for (int i = 1; i < BITS; ++i)
                    if (lane == i) mine = make_uint4(b[i][0], b[i][1], b[i][2], b[i][3]);
                if (lane < BITS)
                    *reinterpret_cast<uint4 *>(planes + (ru * BITS + lane) * (int64_t)kw + seg * 4) = mine;
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

template <int BITS>
void launch_encode(const float *x, int64_t rows, int k, int64_t ldx, float scale, bool relu, uint32_t *planes,
                   int32_t *rowsum, cudaStream_t st) {
    constexpr int UN = 4;
    const float inv2s = 1.0f / (2.0f * scale);
    float lo, hi;
    qnn_clamp_bounds(BITS, scale, relu, &lo, &hi);
    const int kw = (int)qnn_row_words_i(k);
    const int segs = kw / 4;
    int groups;
    int64_t total;                                   // warp-level work items
    const int rpu = (k <= 32) ? 4 : (k <= 64 ? 2 : 1);
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
#define QNN_ENC(RPU_, FULL_)                                                                                       \
    encode_pack_kernel<BITS, UN, RPU_, FULL_><<<grid, kEncThreads, 0, st>>>(x, rows, k, ldx, inv2s, lo, hi, planes, \
                                                                           rowsum, groups, segs, kw, row_step, grp_step)
    if (rpu == 1) {
        if (k % 128 == 0) QNN_ENC(1, true); else QNN_ENC(1, false);
    } else if (rpu == 2) {
        if (k == 64) QNN_ENC(2, true); else QNN_ENC(2, false);
    } else {
        if (k == 32) QNN_ENC(4, true); else QNN_ENC(4, false);
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

extern "C" int qnn_encode_pack(const float *x, int64_t rows, int k, int64_t ldx, int bits, float scale,
                               unsigned flags, uint32_t *planes, int32_t *rowsum, void *stream) {
    if (!x || !planes || rows <= 0 || k <= 0 || ldx < k || !qnn_bits_ok(bits) || (flags & ~QNN_RELU)) return QNN_E_ARG;
    if (!(scale >= 1e-30f) || !(scale <= 1e30f)) return QNN_E_SCALE;   // also rejects NaN, 0, negatives, infinities
    if (!qnn_aligned(planes, 16) || !qnn_aligned(x, 4) || (rowsum && !qnn_aligned(rowsum, 4))) return QNN_E_ALIGN;
    if (k > (1 << 30) || rows > ((int64_t)1 << 40)) return QNN_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const bool relu = (flags & QNN_RELU) != 0;
    if (rowsum && k > 64 && cudaMemsetAsync(rowsum, 0, (size_t)rows * sizeof(int32_t), st) != cudaSuccess)
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

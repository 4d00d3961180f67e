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

template <int BITS>
__global__ void __launch_bounds__(kEncThreads)
encode_pack_kernel(const float *__restrict__ x, int64_t rows, int k, int64_t ldx, float inv2s, bool relu,
                   uint32_t *__restrict__ planes, int32_t *__restrict__ rowsum, int segs_per_row, int kw) {
    const float half = (float)(1 << (BITS - 1));
    const float amax = (float)((1 << BITS) - 1);
    const int lane = threadIdx.x & 31;
    const int64_t warp0 = ((int64_t)blockIdx.x * kEncThreads + threadIdx.x) >> 5;
    const int64_t nwarps = ((int64_t)gridDim.x * kEncThreads) >> 5;
    const int64_t units = rows * segs_per_row;
    for (int64_t u = warp0; u < units; u += nwarps) {
        const int64_t row = u / segs_per_row;
        const int seg = (int)(u - row * segs_per_row);
        const float *src = x + row * ldx;
        const int k0 = seg * 128 + lane;
        float v[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int kk = k0 + 32 * j;
            v[j] = (kk < k) ? __ldcs(src + kk) : 0.0f;
        }
        int t[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            int kk = k0 + 32 * j;
            t[j] = (kk < k) ? qnn_code_t(v[j], inv2s, half, amax, relu) : 0;   // padding bits are 0
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
        if (lane < BITS) {
            uint4 *dst = reinterpret_cast<uint4 *>(planes + (row * BITS + lane) * (int64_t)kw + seg * 4);
            *dst = mine;
        }
        if (rowsum != nullptr) {
            int s = t[0] + t[1] + t[2] + t[3];
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
            if (lane == 0) atomicAdd(rowsum + row, s);
        }
    }
}

// Offline weight packer: one warp per (output feature, group of 4 words).  A word
// covers 32 input channels of one tap; the source index follows the layout flag.
template <int BITS>
__global__ void __launch_bounds__(kEncThreads)
pack_weights_kernel(const float *__restrict__ w, int n_out, int taps, int c_in, int layout, float inv2s,
                    uint32_t *__restrict__ planes, int kw, int cw) {
    const float half = (float)(1 << (BITS - 1));
    const float amax = (float)((1 << BITS) - 1);
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
                t[j] = qnn_code_t(w[idx], inv2s, half, amax, false);
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
void launch_encode(const float *x, int64_t rows, int k, int64_t ldx, float inv2s, bool relu, uint32_t *planes,
                   int32_t *rowsum, cudaStream_t st) {
    const int kw = (int)qnn_row_words_i(k);
    const int segs = kw / 4;
    encode_pack_kernel<BITS><<<grid_for(rows * segs), kEncThreads, 0, st>>>(x, rows, k, ldx, inv2s, relu, planes,
                                                                          rowsum, segs, kw);
}

template <int BITS>
void launch_pack_w(const float *w, int n_out, int taps, int c_in, int layout, float inv2s, uint32_t *planes,
                   cudaStream_t st) {
    const int kw = (int)qnn_w_row_words_i(taps, c_in);
    const int cw = (c_in + 31) / 32;
    pack_weights_kernel<BITS><<<grid_for((int64_t)n_out * (kw / 4)), kEncThreads, 0, st>>>(w, n_out, taps, c_in, layout,
                                                                                      inv2s, planes, kw, cw);
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
    if (!(scale > 0.0f) || !isfinite(scale)) return QNN_E_SCALE;
    if (!qnn_aligned(planes, 16) || !qnn_aligned(x, 4) || (rowsum && !qnn_aligned(rowsum, 4))) return QNN_E_ALIGN;
    if (k > (1 << 30) || rows > ((int64_t)1 << 40)) return QNN_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float inv2s = 1.0f / (2.0f * scale);
    const bool relu = (flags & QNN_RELU) != 0;
    if (rowsum && cudaMemsetAsync(rowsum, 0, (size_t)rows * sizeof(int32_t), st) != cudaSuccess) return QNN_E_CUDA;
#define CALL(B) launch_encode<B>(x, rows, k, ldx, inv2s, relu, planes, rowsum, st)
    QNN_DISPATCH_BITS(bits, CALL)
#undef CALL
    return qnn_launch_status();
}

extern "C" int qnn_pack_weights(const float *w, int n_out, int taps, int c_in, int layout, int bits, float scale,
                                void *packed, void *stream) {
    if (!w || !packed || n_out <= 0 || taps <= 0 || c_in <= 0 || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (layout != QNN_W_NTC && layout != QNN_W_TCN && layout != QNN_W_NCT) return QNN_E_ARG;
    if (!(scale > 0.0f) || !isfinite(scale)) return QNN_E_SCALE;
    if (!qnn_aligned(packed, 16) || !qnn_aligned(w, 4)) return QNN_E_ALIGN;
    const int64_t kw = qnn_w_row_words_i(taps, c_in);
    if (kw > (1 << 26) || (int64_t)n_out * bits * kw > ((int64_t)1 << 40)) return QNN_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const float inv2s = 1.0f / (2.0f * scale);
    uint32_t *planes = static_cast<uint32_t *>(packed);
    int32_t *tapsum = reinterpret_cast<int32_t *>(planes + (int64_t)n_out * bits * kw);
#define CALL(B) launch_pack_w<B>(w, n_out, taps, c_in, layout, inv2s, planes, st)
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

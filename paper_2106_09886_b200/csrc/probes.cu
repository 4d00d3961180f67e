// Peak probes: a register-resident kernel with the contraction's instruction mix, and a plain copy.
#include "qnn_internal.cuh"
#include "bgemm_tiled.cuh"

namespace {

// R x C register tile of xor + popc + add, operands perturbed once per iteration.
template <int R, int C>
__global__ void __launch_bounds__(256) probe_popc_kernel(int iters, int32_t *sink) {
    uint32_t a[R], w[C];
    int acc[R][C];
#pragma unroll
    for (int r = 0; r < R; ++r) a[r] = (threadIdx.x + 1u) * 2654435761u + r * 40503u + blockIdx.x;
#pragma unroll
    for (int c = 0; c < C; ++c) w[c] = (threadIdx.x + 7u) * 2246822519u + c * 2654435769u;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) acc[r][c] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int c = 0; c < C; ++c) acc[r][c] += __popc(a[r] ^ w[c]);
#pragma unroll
        for (int r = 0; r < R; ++r) a[r] += 0x9e3779b9u;
#pragma unroll
        for (int c = 0; c < C; ++c) w[c] += 0x7f4a7c15u;
    }
    int s = 0;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) s += acc[r][c];
    sink[blockIdx.x * 256 + threadIdx.x] = s;
}

// Carry-save form: three xor words are compressed to a sum word and a carry word (two 3-input
// logic ops), so 3 words cost 2 popcounts.
template <int R, int C>
__global__ void __launch_bounds__(256) probe_csa_kernel(int iters, int32_t *sink) {
    uint32_t a[3][R], w[3][C];
    int acc[R][C];
#pragma unroll
    for (int k = 0; k < 3; ++k) {
#pragma unroll
        for (int r = 0; r < R; ++r) a[k][r] = (threadIdx.x + 1u) * 2654435761u + (k * R + r) * 40503u + blockIdx.x;
#pragma unroll
        for (int c = 0; c < C; ++c) w[k][c] = (threadIdx.x + 7u) * 2246822519u + (k * C + c) * 2654435769u;
    }
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) acc[r][c] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int r = 0; r < R; ++r)
#pragma unroll
            for (int c = 0; c < C; ++c) {
                uint32_t x0 = a[0][r] ^ w[0][c], x1 = a[1][r] ^ w[1][c], x2 = a[2][r] ^ w[2][c];
                uint32_t s = x0 ^ x1 ^ x2;
                uint32_t cy = (x0 & x1) | (x2 & (x0 ^ x1));
                acc[r][c] += __popc(s) + 2 * __popc(cy);
            }
#pragma unroll
        for (int k = 0; k < 3; ++k) {
#pragma unroll
            for (int r = 0; r < R; ++r) a[k][r] += 0x9e3779b9u;
#pragma unroll
            for (int c = 0; c < C; ++c) w[k][c] += 0x7f4a7c15u;
        }
    }
    int s = 0;
#pragma unroll
    for (int r = 0; r < R; ++r)
#pragma unroll
        for (int c = 0; c < C; ++c) s += acc[r][c];
    sink[blockIdx.x * 256 + threadIdx.x] = s;
}

// Warp-level 1-bit MMA (m16n8k256), eight independent accumulator tiles per warp, fixed operands.
// XOR = false: and.popc, true: xor.popc.  One instruction is 16*8*256 binary multiply-accumulates.
template <bool XOR>
__global__ void __launch_bounds__(256) probe_bmma_kernel(int iters, int32_t *sink) {
    const uint32_t h = (threadIdx.x + 1u) * 2654435761u + blockIdx.x;
    const uint32_t a0 = h, a1 = h * 2246822519u, a2 = h ^ (h >> 5), a3 = h * 3266489917u, b0 = ~h, b1 = h * 40503u;
    int d[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) d[i][j] = 0;
    for (int it = 0; it < iters; ++it) {
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (XOR)
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                    "{%0,%1,%2,%3};"
                    : "+r"(d[i][0]), "+r"(d[i][1]), "+r"(d[i][2]), "+r"(d[i][3])
                    : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
            else
                asm volatile(
                    "mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
                    "{%0,%1,%2,%3};"
                    : "+r"(d[i][0]), "+r"(d[i][1]), "+r"(d[i][2]), "+r"(d[i][3])
                    : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
        }
    }
    int s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) s += d[i][j];
    sink[blockIdx.x * 256 + threadIdx.x] = s;
}

__global__ void __launch_bounds__(256) probe_copy_kernel(uint4 *__restrict__ dst, const uint4 *__restrict__ src, size_t n) {
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

// The plain fp32 product the efficiency experiment (Section 5.4, Fig. 7) times the bit-plane product against: one
// thread per output element, one multiply-add per step of the reduction, operands straight from global memory, no
// tiling, no shared memory, no tensor cores.  c[m][n] = sum_k a[m][k] * b[k][n], all row-major.
__global__ void __launch_bounds__(256) probe_naive_sgemm_kernel(const float *__restrict__ a, const float *__restrict__ b,
                                                                float *__restrict__ c, int m, int n, int k) {
    const int col = blockIdx.x * 32 + (threadIdx.x & 31);
    const int row = blockIdx.y * 8 + (threadIdx.x >> 5);
    if (row >= m || col >= n) return;
    const float *ar = a + (size_t)row * k;
    float acc = 0.f;
    for (int i = 0; i < k; ++i) acc = fmaf(ar[i], b[(size_t)i * n + col], acc);
    c[(size_t)row * n + col] = acc;
}

}  // namespace

extern "C" int qnn_probe_naive_sgemm(const float *a, const float *b, float *c, int m, int n, int k, void *stream) {
    if (!a || !b || !c || m <= 0 || n <= 0 || k <= 0) return QNN_E_ARG;
    if ((m + 7) / 8 > 65535) return QNN_E_RANGE;
    dim3 grid((n + 31) / 32, (m + 7) / 8);
    probe_naive_sgemm_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(a, b, c, m, n, k);
    return qnn_launch_status();
}

extern "C" int qnn_probe_bitops(int variant, int iters, int blocks, int32_t *sink, double *word_ops, void *stream) {
    if (!sink || iters <= 0 || blocks <= 0 || (variant < 0 || variant > 4)) return QNN_E_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    double per_thread_iter;
    if (variant == 0) {
        probe_popc_kernel<8, 4><<<blocks, 256, 0, st>>>(iters, sink);
        per_thread_iter = 32.0;
    } else if (variant == 1) {
        probe_csa_kernel<4, 4><<<blocks, 256, 0, st>>>(iters, sink);
        per_thread_iter = 48.0;
    } else if (variant == 2) {
        qnn_tiled::probe_csa73_kernel<<<blocks, 256, 0, st>>>(iters, sink);
        per_thread_iter = qnn_tiled::kProbeCsa73WordsPerThreadIter;
    } else {
        if (variant == 3) probe_bmma_kernel<false><<<blocks, 256, 0, st>>>(iters, sink);
        else probe_bmma_kernel<true><<<blocks, 256, 0, st>>>(iters, sink);
        per_thread_iter = 8.0 * 16 * 8 * 256 / 32.0 / 32.0;   // 8 MMAs per warp iteration, in 32-bit word-ops per thread
    }
    if (word_ops) *word_ops = per_thread_iter * iters * 256.0 * blocks;
    return qnn_launch_status();
}

extern "C" int qnn_probe_copy(void *dst, const void *src, size_t bytes, void *stream) {
    if (!dst || !src || bytes == 0 || bytes % 16) return QNN_E_ARG;
    if (!qnn_aligned(dst, 16) || !qnn_aligned(src, 16)) return QNN_E_ALIGN;
    probe_copy_kernel<<<148 * 16, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint4 *>(dst),
                                                                           static_cast<const uint4 *>(src), bytes / 16);
    return qnn_launch_status();
}

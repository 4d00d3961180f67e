// Backward products of a fully-connected layer (Algorithm 1, backward propagation).
//
// With g_hat = alpha * g the two products are dense real-by-integer contractions,
//   G [r][k] = sum_n g_hat[r][n] * qw[n][k]      (g_{a^m} = 2^(m-1) * G,  since sum_j 2^(j-1) W^j = qw)
//   GW[n][k] = sum_r g_hat[r][n] * qa[r][k]      (g_{W^j} = 2^(j-1) * GW, since sum_m 2^(m-1) a^m = qa)
// and run on the tensor cores: one TF32 GEMM C = alpha * A * B^T with both operands K-major in shared memory
// (tcgen05.mma, kind::tf32, accumulator in tensor memory), fed by TMA through a ring of mbarrier-guarded stages.
// The integer codes (|q| <= 255) are exact in TF32; the gradient keeps 11 significant bits per element.
// Bound: tensor pipe (2*M*N*K flop per call).
#include "tc_gemm.cuh"

namespace {

__device__ unsigned int g_tc_error;   // 0 = no error; else 1 + the id of the wait that gave up first

// ------------------------------------------------------------------------------------------------ staging kernels

// Bit planes [rows][bits][kw] -> odd codes q = 2t - (2^bits - 1) as fp32.  TRANSPOSE = false: out[row][col], a
// block covers 32 rows x 256 columns (warp w owns plane word w of eight).  TRANSPOSE = true: out[col][row], a block
// covers 256 rows x 32 columns (one plane word per row), so that each output row receives 1 KiB in one piece.
// The 32 threads of a warp run along the contiguous index of the output: every store instruction writes one line.
template <bool TRANSPOSE, int BITS>
__global__ void __launch_bounds__(256) unpack_codes_kernel(const uint32_t *__restrict__ planes, long long rows, long long k,
                                                          long long kw, float *__restrict__ out, long long ld) {
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const float amax = (float)((1 << BITS) - 1);
    if (TRANSPOSE) {
        const long long row = (long long)blockIdx.y * 256 + threadIdx.x, wcol = blockIdx.x;
        if (row >= rows) return;
        uint32_t w[BITS];
#pragma unroll
        for (int b = 0; b < BITS; ++b) w[b] = __ldg(planes + (row * BITS + b) * kw + wcol);
        const int ncol = (int)min(32ll, k - wcol * 32);
        float *o = out + wcol * 32 * ld + row;
#pragma unroll 8
        for (int c = 0; c < 32; ++c) {
            int t = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) t |= (int)((w[b] >> c) & 1u) << b;
            if (c < ncol) o[c * ld] = (float)(2 * t) - amax;   // default cache policy: the GEMM reads it next, from L2
        }
    } else {
        const long long r0 = (long long)blockIdx.y * 32, wcol = (long long)blockIdx.x * 8 + ty;
        const long long col = wcol * 32 + tx;
        if (wcol * 32 >= k) return;
#pragma unroll 4
        for (int i = 0; i < 32; ++i) {
            const long long row = r0 + i;
            if (row >= rows) break;
            int t = 0;
#pragma unroll
            for (int b = 0; b < BITS; ++b) t |= (int)((__ldg(planes + (row * BITS + b) * kw + wcol) >> tx) & 1u) << b;
            if (col < k) out[row * ld + col] = (float)(2 * t) - amax;
        }
    }
}

// out[c][r] = in[r][c] through a 32 x 33 shared tile (both sides coalesced).
__global__ void __launch_bounds__(256) transpose_f32_kernel(const float *__restrict__ in, long long rows, long long cols,
                                                           long long ld_in, float *__restrict__ out, long long ld_out) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const long long r0 = (long long)blockIdx.y * 32, c0 = (long long)blockIdx.x * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long r = r0 + ty + 8 * i, c = c0 + tx;
        tile[ty + 8 * i][tx] = (r < rows && c < cols) ? in[r * ld_in + c] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long c = c0 + ty + 8 * i, r = r0 + tx;
        if (c < cols && r < rows) out[c * ld_out + r] = tile[tx][ty + 8 * i];
    }
}

// Row-padded copy for a gradient whose rows are not 16-byte multiples (TMA needs them to be).
__global__ void __launch_bounds__(256) copy_rows_kernel(const float *__restrict__ in, long long rows, long long cols,
                                                       float *__restrict__ out, long long ld_out) {
    const long long total = rows * cols;
    for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < total; i += (long long)gridDim.x * blockDim.x)
        out[(i / cols) * ld_out + i % cols] = in[i];
}

template <bool TRANSPOSE>
void launch_unpack(const uint32_t *planes, long long rows, long long k, int bits, long long kw, float *out, long long ld,
                   cudaStream_t st) {
    const dim3 grid = TRANSPOSE ? dim3((unsigned)qnn_ceil_div(k, 32), (unsigned)qnn_ceil_div(rows, 256))
                                : dim3((unsigned)qnn_ceil_div(k, 256), (unsigned)qnn_ceil_div(rows, 32));
#define UNPACK_CASE(B) case B: unpack_codes_kernel<TRANSPOSE, B><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    switch (bits) {
        UNPACK_CASE(1) UNPACK_CASE(2) UNPACK_CASE(3) UNPACK_CASE(4) UNPACK_CASE(5) UNPACK_CASE(6) UNPACK_CASE(7)
        default: unpack_codes_kernel<TRANSPOSE, 8><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    }
#undef UNPACK_CASE
}

int unpack_codes(const uint32_t *planes, long long rows, long long k, int bits, bool transpose, float *out, long long ld,
                 cudaStream_t st) {
    const long long kw = qnn_row_words_i(k);
    if (transpose) launch_unpack<true>(planes, rows, k, bits, kw, out, ld, st);
    else launch_unpack<false>(planes, rows, k, bits, kw, out, ld, st);
    return qnn_launch_status();
}

}  // namespace

// Device address of the word in which a tensor-path kernel of any translation unit records a wait that gave up.
unsigned int *qnn_tc_error_word() {
    void *ptr = nullptr;
    return cudaGetSymbolAddress(&ptr, g_tc_error) == cudaSuccess ? static_cast<unsigned int *>(ptr) : nullptr;
}

// ------------------------------------------------------------------------------------------------ C ABI

static const size_t DIM_LIMIT = (size_t)65535 * 32;   // every dimension may become the y extent of a staging grid

static bool backward_dims_ok(size_t m, size_t n, size_t k) {
    return m >= 1 && n >= 1 && k >= 1 && m <= DIM_LIMIT && n <= DIM_LIMIT && k <= DIM_LIMIT;
}

extern "C" int qnn_unpack_codes_f32(const uint32_t *planes, size_t rows, size_t k, int bits, int transpose, float *out,
                                    size_t ld, void *stream) {
    if (!planes || !out || rows < 1 || k < 1 || rows > DIM_LIMIT || k > DIM_LIMIT || !qnn_bits_ok(bits)) return QNN_E_ARG;
    if (ld < (transpose ? rows : k)) return QNN_E_ARG;
    if (!qnn_aligned(planes, 16) || !qnn_aligned(out, 4)) return QNN_E_ALIGN;
    return unpack_codes(planes, (long long)rows, (long long)k, bits, transpose != 0, out, (long long)ld,
                        static_cast<cudaStream_t>(stream));
}

extern "C" size_t qnn_bgemm_backward_data_workspace(size_t m, size_t n, size_t k) {
    if (!backward_dims_ok(m, n, k)) return 0;
    const size_t ldn = (size_t)pad32((long long)n);
    return (k + (n % 4 ? m : 0)) * ldn * sizeof(float);
}

extern "C" int qnn_bgemm_backward_data(const float *g, const uint32_t *w_planes, size_t m, size_t n, size_t k, int wb,
                                       float alpha, const float *x, int ab, float r, float *out, void *workspace,
                                       size_t workspace_bytes, void *stream) {
    if (!g || !w_planes || !out || !workspace || !backward_dims_ok(m, n, k) || !qnn_bits_ok(wb)) return QNN_E_ARG;
    if (x && !qnn_bits_ok(ab)) return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (x && (!(r >= 1e-30f) || !(r <= 1e30f))) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bgemm_backward_data_workspace(m, n, k)) return QNN_E_ARG;
    if (!qnn_aligned(g, 16) || !qnn_aligned(w_planes, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(out, 4) ||
        (x && !qnn_aligned(x, 4)))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ldn = pad32((long long)n);
    float *wqt = static_cast<float *>(workspace);                       // [k][ldn]: wqt[kk][nn] = qw[nn][kk]
    int rc = unpack_codes(w_planes, (long long)n, (long long)k, wb, true, wqt, ldn, st);
    if (rc != QNN_OK) return rc;
    const float *a = g;
    long long lda = (long long)n;
    if (n % 4) {                                                        // rows of g are not 16-byte multiples
        float *gp = wqt + (size_t)k * ldn;
        copy_rows_kernel<<<148 * 8, 256, 0, st>>>(g, (long long)m, (long long)n, gp, ldn);
        if ((rc = qnn_launch_status()) != QNN_OK) return rc;
        a = gp;
        lda = ldn;
    }
    GemmParams p{};
    p.M = (int)m; p.N = (int)k; p.K = (int)n;
    p.alpha = alpha;
    p.C = out; p.ldc = (long long)k;
    p.x = x; p.ldx = (long long)k; p.bits = ab; p.r = r;
    if (x) p.enc = mbit_plane_consts(ab);
    if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
    return run_gemm<TC_TF32>(a, lda, wqt, ldn, p, st);
}

extern "C" size_t qnn_bgemm_backward_weights_workspace(size_t m, size_t n, size_t k) {
    if (!backward_dims_ok(m, n, k)) return 0;
    return (n + k) * (size_t)pad32((long long)m) * sizeof(float);
}

extern "C" int qnn_bgemm_backward_weights(const float *g, const uint32_t *a_planes, size_t m, size_t n, size_t k, int ab,
                                          float alpha, float *gw, void *workspace, size_t workspace_bytes, void *stream) {
    if (!g || !a_planes || !gw || !workspace || !backward_dims_ok(m, n, k) || !qnn_bits_ok(ab)) return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bgemm_backward_weights_workspace(m, n, k)) return QNN_E_ARG;
    if (!qnn_aligned(g, 4) || !qnn_aligned(a_planes, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(gw, 4))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ldm = pad32((long long)m);
    float *gt = static_cast<float *>(workspace);                        // [n][ldm]: gt[nn][rr] = g[rr][nn]
    float *aqt = gt + (size_t)n * ldm;                                  // [k][ldm]: aqt[kk][rr] = qa[rr][kk]
    const dim3 grid((unsigned)qnn_ceil_div((long long)n, 32), (unsigned)qnn_ceil_div((long long)m, 32));
    transpose_f32_kernel<<<grid, 256, 0, st>>>(g, (long long)m, (long long)n, (long long)n, gt, ldm);
    int rc = qnn_launch_status();
    if (rc != QNN_OK) return rc;
    if ((rc = unpack_codes(a_planes, (long long)m, (long long)k, ab, true, aqt, ldm, st)) != QNN_OK) return rc;
    GemmParams p{};
    p.M = (int)n; p.N = (int)k; p.K = (int)m;
    p.alpha = alpha;
    p.C = gw; p.ldc = (long long)k;
    if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
    return run_gemm<TC_TF32>(gt, ldm, aqt, ldm, p, st);
}

extern "C" int qnn_tensor_path_status(unsigned int *status) {
    if (!status) return QNN_E_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return QNN_E_CUDA;
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(v)) != cudaSuccess) return QNN_E_CUDA;
    if (v && cudaMemcpyToSymbol(g_tc_error, &zero, sizeof(zero)) != cudaSuccess) return QNN_E_CUDA;
    *status = v;
    return v ? QNN_E_DEVICE : QNN_OK;
}

// Backward products of a fully-connected and of a convolution layer (Algorithm 1, backward propagation).
//
// With g_hat = alpha * g the two products are dense real-by-integer contractions,
//   G [r][k] = sum_n g_hat[r][n] * qw[n][k]      (g_{a^m} = 2^(m-1) * G,  since sum_j 2^(j-1) W^j = qw)
//   GW[n][k] = sum_r g_hat[r][n] * qa[r][k]      (g_{W^j} = 2^(j-1) * GW, since sum_m 2^(m-1) a^m = qa)
// and run on the tensor cores: one TF32 GEMM C = alpha * A * B^T with both operands K-major in shared memory
// (tcgen05.mma, kind::tf32, accumulator in tensor memory), fed by TMA through a ring of mbarrier-guarded stages.
// The integer codes (|q| <= 255) are exact in TF32; the gradient keeps 11 significant bits per element.
// Bound: tensor pipe (2*M*N*K flop per call).
// A convolution goes through the same GEMM: the weight gradient contracts g with the im2col of the activation codes
// (unpacked straight from the planes into K-major order); the data gradient is an implicit GEMM over (tap, output
// feature) whose A operand the TMA unit gathers from g itself, one shifted 4-D box per tap (see ConvGather in
// tc_gemm.cuh), so no patch matrix exists and every result pixel is one fp32 accumulation in tensor memory.
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


// ------------------------------------------------------------------------------------------------ convolution staging

struct ConvGeom {
    int N, H, W, C, Cout, R, S, stride, pad, Ho, Wo, cw;   // cw = ceil(C / 32) words per pixel (tap) and plane
    long long Mg, Kg;                                      // N*Ho*Wo output pixels, R*S*C reduction length
};

// im2col of the activation codes, transposed: colt[(tap*C + c)][m] = qa[n][ho*st - pad + r][wo*st - pad + s][c] for
// output pixel m = (n, ho, wo) and tap = r*S + s, 0 where the tap falls outside the image (the encoded tensor is
// padded with true zeros).  One thread per output pixel and (tap, channel word): it reads the pixel's plane words
// once and writes 32 channels; the 32 threads of a warp are consecutive pixels, so every store writes one line.
template <int BITS>
__global__ void __launch_bounds__(256) conv_codes_t_kernel(const uint32_t *__restrict__ planes, long long a_pitch, ConvGeom g,
                                                          float *__restrict__ colt, long long ld) {
    const long long m = (long long)blockIdx.x * 256 + threadIdx.x;
    if (m >= g.Mg) return;
    const int tap = blockIdx.y / g.cw, cwi = blockIdx.y % g.cw;
    const int r = tap / g.S, sx = tap % g.S;
    const int wo = (int)(m % g.Wo), ho = (int)((m / g.Wo) % g.Ho);
    const long long n = m / ((long long)g.Wo * g.Ho);
    const int hi = ho * g.stride - g.pad + r, wi = wo * g.stride - g.pad + sx;
    const bool inside = hi >= 0 && hi < g.H && wi >= 0 && wi < g.W;
    uint32_t w[BITS];
#pragma unroll
    for (int b = 0; b < BITS; ++b)
        w[b] = inside ? __ldg(planes + (((n * g.H + hi) * g.W + wi) * BITS + b) * a_pitch + cwi) : 0u;
    const float amax = (float)((1 << BITS) - 1);
    const int ncol = min(32, g.C - cwi * 32);
    float *o = colt + ((long long)tap * g.C + cwi * 32) * ld + m;
#pragma unroll 8
    for (int c = 0; c < 32; ++c) {
        int t = 0;
#pragma unroll
        for (int b = 0; b < BITS; ++b) t |= (int)((w[b] >> c) & 1u) << b;
        if (c < ncol) o[c * ld] = inside ? (float)(2 * t) - amax : 0.0f;
    }
}

// Packed convolution weights [Cout][bits][w_pitch] (tap-major words, each tap on a word boundary) -> codes transposed:
// wqt[(tap*C + c)][co] = qw[co][tap][c].  One thread per output feature and (tap, channel word).
template <int BITS>
__global__ void __launch_bounds__(256) conv_weights_t_kernel(const uint32_t *__restrict__ wp, long long w_pitch, ConvGeom g,
                                                            float *__restrict__ wqt, long long ld) {
    const int co = blockIdx.x * 256 + threadIdx.x;
    if (co >= g.Cout) return;
    const int tap = blockIdx.y / g.cw, cwi = blockIdx.y % g.cw;
    uint32_t w[BITS];
#pragma unroll
    for (int b = 0; b < BITS; ++b) w[b] = __ldg(wp + ((long long)co * BITS + b) * w_pitch + (long long)tap * g.cw + cwi);
    const float amax = (float)((1 << BITS) - 1);
    const int ncol = min(32, g.C - cwi * 32);
    float *o = wqt + ((long long)tap * g.C + cwi * 32) * ld + co;
#pragma unroll 8
    for (int c = 0; c < 32; ++c) {
        int t = 0;
#pragma unroll
        for (int b = 0; b < BITS; ++b) t |= (int)((w[b] >> c) & 1u) << b;
        if (c < ncol) o[c * ld] = (float)(2 * t) - amax;
    }
}

// Gradient image g[n][ho][wo][co] -> gt[co][n][ho][wp] (pixel-contiguous, rows padded with zeros from Wo to Wp columns):
// the K-major A operand of the implicit weight gradient.  One block = 32 features x 32 columns of one image row, through
// a 32 x 33 shared tile (both sides coalesced).
__global__ void __launch_bounds__(256) conv_g_t_kernel(const float *__restrict__ g, int Cout, int Wo, long long Wp,
                                                      long long rows /* N*Ho */, float *__restrict__ gt) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const long long row = blockIdx.x;
    const int c0 = blockIdx.y * 32, w0 = blockIdx.z * 32;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int wo = w0 + ty + 8 * i, co = c0 + tx;
        tile[ty + 8 * i][tx] = (wo < Wo && co < Cout) ? g[(row * Wo + wo) * Cout + co] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int co = c0 + ty + 8 * i;
        const long long wp = w0 + tx;
        if (co < Cout && wp < Wp) gt[((long long)co * rows + row) * Wp + wp] = tile[tx][ty + 8 * i];
    }
}

// Activation planes -> the copies of the transposed codes that the implicit weight gradient reads (ConvWeightGather):
// qas[s*st + rho][c][n][a'][j] = qa[n][(a' + qmin)*st + rho][j*st - pad + s][c] where that pixel is inside the image and
// j < Wo, else 0; a' = 0 .. Hq - 1, j = 0 .. Wq - 1.  One thread per (n, a', four consecutive j) and (copy, channel word):
// consecutive threads write consecutive j.
template <int BITS>
__global__ void __launch_bounds__(256) conv_codes_shift_kernel(const uint32_t *__restrict__ planes, long long a_pitch, ConvGeom g,
                                                              int Hq, int Wq, int qmin, float *__restrict__ qas) {
    // four consecutive j per thread (Wq is a multiple of 4): every store is 16 bytes, a warp writes 512 contiguous bytes
    const int wq4 = Wq >> 2;
    const long long idx4 = (long long)blockIdx.x * 256 + threadIdx.x;
    const long long rows_total = (long long)g.N * Hq;
    if (idx4 >= rows_total * wq4) return;
    const long long row = idx4 / wq4;                     // (n, a')
    const int j0 = (int)(idx4 - row * wq4) * 4;
    const long long n = row / Hq;
    const int copy = blockIdx.y / g.cw, cwi = blockIdx.y % g.cw;
    const int s = copy / g.stride, rho = copy - s * g.stride;
    const int h = ((int)(row - n * Hq) + qmin) * g.stride + rho;
    const bool row_inside = h >= 0 && h < g.H;
    uint32_t w[4][BITS];
    bool inside[4];
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int j = j0 + k, wi = j * g.stride - g.pad + s;
        inside[k] = row_inside && j < g.Wo && wi >= 0 && wi < g.W;
#pragma unroll
        for (int b = 0; b < BITS; ++b)
            w[k][b] = inside[k] ? __ldg(planes + (((n * g.H + h) * g.W + wi) * BITS + b) * a_pitch + cwi) : 0u;
    }
    // code 2t - amax as a float without a conversion: the bits of 2^23 + 2t, minus (2^23 + amax); both exact
    const float bias = 8388608.0f + (float)((1 << BITS) - 1);
    const int ncol = min(32, g.C - cwi * 32);
    const long long cstride = rows_total * Wq;
    float *o = qas + ((long long)copy * g.C + cwi * 32) * cstride + row * Wq + j0;
#pragma unroll 4
    for (int c = 0; c < 32; ++c) {
        float v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            uint32_t t2 = 0u;
#pragma unroll
            for (int b = 0; b < BITS; ++b) t2 |= ((w[k][b] >> c) & 1u) << (b + 1);
            v[k] = inside[k] ? __int_as_float((int)(0x4B000000u | t2)) - bias : 0.0f;
        }
        if (c < ncol) *reinterpret_cast<float4 *>(o + c * cstride) = make_float4(v[0], v[1], v[2], v[3]);
    }
}

bool conv_geom(int N, int H, int W, int C, int Cout, int R, int S, int stride, int pad, ConvGeom *g) {
    if (N < 1 || H < 1 || W < 1 || C < 1 || Cout < 1 || R < 1 || S < 1 || stride < 1 || pad < 0) return false;
    const long long Ho = ((long long)H + 2 * pad - R) / stride + 1, Wo = ((long long)W + 2 * pad - S) / stride + 1;
    if ((long long)H + 2 * pad < R || (long long)W + 2 * pad < S || Ho < 1 || Wo < 1) return false;
    g->N = N; g->H = H; g->W = W; g->C = C; g->Cout = Cout; g->R = R; g->S = S; g->stride = stride; g->pad = pad;
    g->Ho = (int)Ho; g->Wo = (int)Wo; g->cw = (C + 31) / 32;
    g->Mg = (long long)N * Ho * Wo;
    g->Kg = (long long)R * S * C;
    return true;
}

size_t round256(size_t v) { return (v + 255) / 256 * 256; }

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
    return (n + k) * (size_t)pad32((long long)m) * sizeof(float) + gemm_split_workspace((long long)n, (long long)k, (long long)m);
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
    // a small n x k result against a long batch: the contraction over the batch is split over the CTAs
    return run_gemm_tf32_split(gt, ldm, aqt, ldm, p, aqt + (size_t)k * ldm, st);
}


// ------------------------------------------------------------------------------------------------ convolution backward

static bool conv_backward_dims_ok(const ConvGeom &g) {
    return g.Mg <= (long long)DIM_LIMIT && g.Kg <= (long long)DIM_LIMIT && (size_t)g.Cout <= DIM_LIMIT &&
           (long long)g.R * g.S * g.cw <= 65535 && (long long)g.N * g.H * g.W <= (1ll << 40);
}

extern "C" size_t qnn_bconv2d_backward_data_workspace(int N, int H, int W, int C, int Cout, int R, int S, int stride, int pad) {
    ConvGeom g;
    if (!conv_geom(N, H, W, C, Cout, R, S, stride, pad, &g) || !conv_backward_dims_ok(g)) return 0;
    const size_t ldn = (size_t)pad32(Cout);
    return round256((size_t)g.Kg * ldn * 4) + (Cout % 4 ? round256((size_t)g.Mg * ldn * 4) : 0);
}

extern "C" int qnn_bconv2d_backward_data(const float *g, const void *w_packed, int wb, int N, int H, int W, int C, int Cout,
                                         int R, int S, int stride, int pad, float alpha, const float *x, int ab, float r,
                                         float *out, void *workspace, size_t workspace_bytes, void *stream) {
    ConvGeom cg;
    if (!g || !w_packed || !out || !workspace || !qnn_bits_ok(wb) || !conv_geom(N, H, W, C, Cout, R, S, stride, pad, &cg) ||
        !conv_backward_dims_ok(cg))
        return QNN_E_ARG;
    if (x && !qnn_bits_ok(ab)) return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (x && (!(r >= 1e-30f) || !(r <= 1e30f))) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bconv2d_backward_data_workspace(N, H, W, C, Cout, R, S, stride, pad)) return QNN_E_ARG;
    if (!qnn_aligned(g, 16) || !qnn_aligned(w_packed, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(out, 4) ||
        (x && !qnn_aligned(x, 4)))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ldn = pad32(Cout);
    char *ws = static_cast<char *>(workspace);
    float *wqt = reinterpret_cast<float *>(ws);                         // [Kg][ldn]
    ws += round256((size_t)cg.Kg * ldn * 4);
    const dim3 wgrid((unsigned)qnn_ceil_div(Cout, 256), (unsigned)(R * S * cg.cw));
    const long long w_pitch = qnn_w_row_words_i(R * S, C);
#define CONV_W_CASE(B) case B: conv_weights_t_kernel<B><<<wgrid, 256, 0, st>>>(static_cast<const uint32_t *>(w_packed), w_pitch, cg, wqt, ldn); break;
    switch (wb) {
        CONV_W_CASE(1) CONV_W_CASE(2) CONV_W_CASE(3) CONV_W_CASE(4) CONV_W_CASE(5) CONV_W_CASE(6) CONV_W_CASE(7)
        default: conv_weights_t_kernel<8><<<wgrid, 256, 0, st>>>(static_cast<const uint32_t *>(w_packed), w_pitch, cg, wqt, ldn); break;
    }
#undef CONV_W_CASE
    int rc = qnn_launch_status();
    if (rc != QNN_OK) return rc;
    const float *a = g;
    long long lda = Cout;
    if (Cout % 4) {                                                     // rows of g are not 16-byte multiples
        float *gp = reinterpret_cast<float *>(ws);
        ws += round256((size_t)cg.Mg * ldn * 4);
        copy_rows_kernel<<<148 * 8, 256, 0, st>>>(g, cg.Mg, (long long)Cout, gp, ldn);
        if ((rc = qnn_launch_status()) != QNN_OK) return rc;
        a = gp;
        lda = ldn;
    }
    GemmParams p{};
    p.alpha = alpha;
    p.C = out; p.ldc = C;
    p.x = x; p.ldx = C; p.bits = ab; p.r = r;
    if (x) p.enc = mbit_plane_consts(ab);
    if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
    // implicit gather: the tensor cores read shifted boxes of g and the tap's weight codes; no patch matrix
    return run_conv_data_gradient(a, lda, wqt, ldn, N, H, W, C, Cout, R, S, stride, pad, cg.Ho, cg.Wo, p, st);
}

// The weight gradient runs as an implicit GEMM on the transposed gradient and S*stride copies of the transposed codes
// (ConvWeightGather) where those copies are clearly smaller than the R*S-fold patch matrix; otherwise, and for
// geometries beyond the index ranges below, it stages the whole patch matrix.
static bool wgrad_implicit(const ConvGeom &g) {
    const ConvWgradPlan pl = conv_wgrad_plan(g.N, g.C, g.Cout, g.R, g.S, g.stride, g.pad, g.Ho, g.Wo);
    const long long Wq = pl.Wq, Hq = pl.Hq, copies = (long long)g.S * g.stride;
    // worth it when the copies are clearly smaller than the patch matrix: always at stride 1 (3 x 3: 0.4 of it); at
    // stride 2 a 3 x 3 kernel's six half-height copies are 0.8 of it and measured 12% slower, so those stay explicit
    if (4 * copies * Hq * Wq > 3ll * g.R * g.S * g.Ho * g.Wo) return false;
    return g.stride <= 16 && (long long)g.N * g.Ho <= 0x7FFFFFFFll && Wq <= 65535 * 32 && copies * g.cw <= 65535 &&
           (long long)g.N * Hq * Wq <= (1ll << 36) && Wq * Hq * g.N * (long long)g.C * copies < (1ll << 37) &&
           Wq * g.Ho * g.N * (long long)g.Cout < (1ll << 36);
}

extern "C" size_t qnn_bconv2d_backward_weights_workspace(int N, int H, int W, int C, int Cout, int R, int S, int stride,
                                                         int pad) {
    ConvGeom g;
    if (!conv_geom(N, H, W, C, Cout, R, S, stride, pad, &g) || !conv_backward_dims_ok(g)) return 0;
    if (wgrad_implicit(g)) {
        const ConvWgradPlan pl = conv_wgrad_plan(N, C, Cout, R, S, stride, pad, g.Ho, g.Wo);
        return round256((size_t)Cout * N * g.Ho * pl.Wq * 4) + round256((size_t)S * stride * C * N * pl.Hq * pl.Wq * 4) +
               round256(conv_wgrad_split_workspace(N, C, Cout, R, S, stride, pad, g.Ho, g.Wo));
    }
    const size_t ldm = (size_t)pad32(g.Mg);
    return round256((size_t)Cout * ldm * 4) + round256((size_t)g.Kg * ldm * 4) + round256(gemm_split_workspace(Cout, g.Kg, g.Mg));
}

extern "C" int qnn_bconv2d_backward_weights(const float *g, const uint32_t *a_planes, int ab, int N, int H, int W, int C,
                                            int Cout, int R, int S, int stride, int pad, float alpha, float *gw,
                                            void *workspace, size_t workspace_bytes, void *stream) {
    ConvGeom cg;
    if (!g || !a_planes || !gw || !workspace || !qnn_bits_ok(ab) || !conv_geom(N, H, W, C, Cout, R, S, stride, pad, &cg) ||
        !conv_backward_dims_ok(cg))
        return QNN_E_ARG;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bconv2d_backward_weights_workspace(N, H, W, C, Cout, R, S, stride, pad)) return QNN_E_ARG;
    if (!qnn_aligned(g, 4) || !qnn_aligned(a_planes, 16) || !qnn_aligned(workspace, 256) || !qnn_aligned(gw, 4))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (wgrad_implicit(cg)) {
        const ConvWgradPlan pl = conv_wgrad_plan(N, C, Cout, R, S, stride, pad, cg.Ho, cg.Wo);
        const long long Wq = pl.Wq, Hq = pl.Hq, rows = (long long)N * cg.Ho, copies = (long long)S * stride;
        float *gt = static_cast<float *>(workspace);                    // [Cout][N][Ho][Wq]
        float *qas = reinterpret_cast<float *>(static_cast<char *>(workspace) + round256((size_t)Cout * rows * Wq * 4));   // [S*stride][C][N][Hq][Wq]
        void *split_ws = reinterpret_cast<char *>(qas) + round256((size_t)copies * C * N * Hq * Wq * 4);
        if (Wq == cg.Wo && qnn_ceil_div(cg.Mg, 32) <= 65535) {
            // no row padding: gt[co][pixel] is the plain transpose of g[pixel][co], whole 32 x 32 tiles throughout
            const dim3 tgrid((unsigned)qnn_ceil_div(Cout, 32), (unsigned)qnn_ceil_div(cg.Mg, 32));
            transpose_f32_kernel<<<tgrid, 256, 0, st>>>(g, cg.Mg, (long long)Cout, (long long)Cout, gt, cg.Mg);
        } else {
            const dim3 ggrid((unsigned)rows, (unsigned)qnn_ceil_div(Cout, 32), (unsigned)qnn_ceil_div(Wq, 32));
            conv_g_t_kernel<<<ggrid, 256, 0, st>>>(g, Cout, cg.Wo, Wq, rows, gt);
        }
        int rc = qnn_launch_status();
        if (rc != QNN_OK) return rc;
        const dim3 sgrid((unsigned)qnn_ceil_div((long long)N * Hq * (Wq / 4), 256), (unsigned)(copies * cg.cw));
        const long long a_pitch = qnn_row_words_i(C);
#define CONV_S_CASE(B) case B: conv_codes_shift_kernel<B><<<sgrid, 256, 0, st>>>(a_planes, a_pitch, cg, (int)Hq, (int)Wq, pl.qmin, qas); break;
        switch (ab) {
            CONV_S_CASE(1) CONV_S_CASE(2) CONV_S_CASE(3) CONV_S_CASE(4) CONV_S_CASE(5) CONV_S_CASE(6) CONV_S_CASE(7)
            default: conv_codes_shift_kernel<8><<<sgrid, 256, 0, st>>>(a_planes, a_pitch, cg, (int)Hq, (int)Wq, pl.qmin, qas); break;
        }
#undef CONV_S_CASE
        if ((rc = qnn_launch_status()) != QNN_OK) return rc;
        GemmParams p{};
        p.alpha = alpha;
        p.C = gw; p.ldc = cg.Kg;
        if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
        return run_conv_weight_gradient(gt, qas, N, C, Cout, R, S, stride, pad, cg.Ho, cg.Wo, p, split_ws, st);
    }
    const long long ldm = pad32(cg.Mg);
    float *gt = static_cast<float *>(workspace);                        // [Cout][ldm]: gt[co][m] = g[m][co]
    float *colt = reinterpret_cast<float *>(static_cast<char *>(workspace) + round256((size_t)Cout * ldm * 4));   // [Kg][ldm]
    const dim3 tgrid((unsigned)qnn_ceil_div(Cout, 32), (unsigned)qnn_ceil_div(cg.Mg, 32));
    transpose_f32_kernel<<<tgrid, 256, 0, st>>>(g, cg.Mg, (long long)Cout, (long long)Cout, gt, ldm);
    int rc = qnn_launch_status();
    if (rc != QNN_OK) return rc;
    const dim3 cgrid((unsigned)qnn_ceil_div(cg.Mg, 256), (unsigned)(R * S * cg.cw));
    const long long a_pitch = qnn_row_words_i(C);
#define CONV_A_CASE(B) case B: conv_codes_t_kernel<B><<<cgrid, 256, 0, st>>>(a_planes, a_pitch, cg, colt, ldm); break;
    switch (ab) {
        CONV_A_CASE(1) CONV_A_CASE(2) CONV_A_CASE(3) CONV_A_CASE(4) CONV_A_CASE(5) CONV_A_CASE(6) CONV_A_CASE(7)
        default: conv_codes_t_kernel<8><<<cgrid, 256, 0, st>>>(a_planes, a_pitch, cg, colt, ldm); break;
    }
#undef CONV_A_CASE
    if ((rc = qnn_launch_status()) != QNN_OK) return rc;
    GemmParams p{};
    p.M = Cout; p.N = (int)cg.Kg; p.K = (int)cg.Mg;
    p.alpha = alpha;
    p.C = gw; p.ldc = cg.Kg;
    if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
    // few output tiles (Cout x R*S*C) against a contraction over every output pixel: split it over the CTAs
    void *split_ws = reinterpret_cast<char *>(colt) + round256((size_t)cg.Kg * ldm * 4);
    return run_gemm_tf32_split(gt, ldm, colt, ldm, p, split_ws, st);
}

// ------------------------------------------------------------------------------------------------ wait self-test

namespace {

__device__ __align__(128) uint32_t g_selftest_src[32];      // source of the self-test's bulk copy (contents irrelevant)

// One CTA, two warps, built from the same helpers as tc_gemm_kernel so that their give-up path runs once on demand:
//   warp 0, lane 0 (producer role): starts one 128-byte bulk copy into shared memory under full[0], then waits for a
//     stage release on empty[0] that no consumer ever gives -> gives up after `limit` polls, raises the CTA's abort
//     flag and the library's error word (wait id 0), and drains its copy in flight like the GEMM's producer;
//   warp 1 (epilogue role): waits, all lanes, for an accumulator on acc_full that no MMA ever commits, with a limit
//     64 times longer, and leaves through the abort flag (or by its own limit).
// Every loop is bounded; the kernel ends normally.
__global__ void __launch_bounds__(64, 1) bounded_wait_selftest_kernel(unsigned int limit, unsigned int *err) {
    __shared__ __align__(128) uint32_t dst[32];
    __shared__ __align__(8) uint64_t bars[3];               // full[0], empty[0], acc_full[0]
    __shared__ uint32_t abort_word;
    volatile uint32_t *abort_flag = &abort_word;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        mbar_init(&bars[0], 1);
        mbar_init(&bars[1], 1);
        mbar_init(&bars[2], 1);
        abort_word = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (warp == 0) {
        if (lane == 0) {
            mbar_expect_tx(&bars[0], 128);
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], 128, [%2];"
                         ::"r"(smem_u32(dst)), "l"(__cvta_generic_to_global(g_selftest_src)), "r"(smem_u32(&bars[0])) : "memory");
            // second use of a one-stage ring: wants the consumer's release of the first use, which never comes
            if (!mbar_wait(&bars[1], 0u, abort_flag, 0, err, limit)) drain_copies_in_flight(&bars[0], 1, 1, limit << 6);
        }
    } else {
        __all_sync(0xffffffffu, mbar_wait(&bars[2], 0u, abort_flag, 2, err, limit << 6));
    }
    __syncthreads();
}

}  // namespace

extern "C" int qnn_selftest_bounded_wait(unsigned int poll_limit, void *stream) {
    if (poll_limit < 16u || poll_limit > (1u << 16)) return QNN_E_ARG;
    unsigned int *err = qnn_tc_error_word();
    if (!err) return QNN_E_CUDA;
    bounded_wait_selftest_kernel<<<1, 64, 0, static_cast<cudaStream_t>(stream)>>>(poll_limit, err);
    return qnn_launch_status();
}

extern "C" int qnn_last_device_status(unsigned int *status) { return qnn_tensor_path_status(status); }

extern "C" int qnn_tensor_path_status(unsigned int *status) {
    if (!status) return QNN_E_ARG;
    if (cudaDeviceSynchronize() != cudaSuccess) return QNN_E_CUDA;
    unsigned int v = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(v)) != cudaSuccess) return QNN_E_CUDA;
    if (v && cudaMemcpyToSymbol(g_tc_error, &zero, sizeof(zero)) != cudaSuccess) return QNN_E_CUDA;
    *status = v;
    return v ? QNN_E_DEVICE : QNN_OK;
}

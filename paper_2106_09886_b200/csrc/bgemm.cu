// qnn_bgemm / qnn_bconv2d: all plane-pair xor+popcount contractions of one layer,
// the 2^(i+j) combine and the scale, in one launch.
#include "qnn_internal.cuh"
#include "bgemm_tiled.cuh"
#include "bconv_dense.cuh"
#include "bconv_pointwise.cuh"

namespace {

struct ConvGeom {
    int N, H, W, C, Cout, R, S, stride, pad, Ho, Wo;
    int cw;        // words per tap: ceil(C/32)
    int a_pitch;   // words per (pixel, plane) in the activation planes: qnn_row_words(C)
    int w_pitch;   // words per (feature, plane) in the packed weights
};

__device__ __forceinline__ void store_out(float *out, int64_t ldo, int32_t *acc, int64_t m, int n, int Ng, int32_t v,
                                          float alpha) {
    if (acc) acc[m * Ng + n] = v;
    if (out) out[m * ldo + n] = __fmul_rn(__int2float_rn(v), alpha);
}

// ---------------------------------------------------------------------------------------------
// Fallback convolution (any ab, wb in 1..8): one thread per output.  Only used for geometries outside the
// tiled kernel's index arithmetic (more than 4095 reduction words per plane, very wide kernels); not tuned.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
bconv_generic_kernel(const uint32_t *__restrict__ a, int ab, const uint32_t *__restrict__ w, int wb, ConvGeom g,
                     float alpha, float *__restrict__ out, int32_t *__restrict__ acc) {
    const int co = blockIdx.x * 16 + (threadIdx.x & 15);
    const int64_t m = (int64_t)blockIdx.y * 16 + (threadIdx.x >> 4);
    const int64_t Mg = (int64_t)g.N * g.Ho * g.Wo;
    if (co >= g.Cout || m >= Mg) return;
    const int wo = (int)(m % g.Wo);
    const int ho = (int)((m / g.Wo) % g.Ho);
    const int n = (int)(m / ((int64_t)g.Wo * g.Ho));
    int32_t s = 0;
    int valid = 0;
    for (int r = 0; r < g.R; ++r) {
        const int hi = ho * g.stride - g.pad + r;
        if (hi < 0 || hi >= g.H) continue;
        for (int t = 0; t < g.S; ++t) {
            const int wi = wo * g.stride - g.pad + t;
            if (wi < 0 || wi >= g.W) continue;
            ++valid;
            const uint32_t *ap = a + (((int64_t)n * g.H + hi) * g.W + wi) * ab * g.a_pitch;
            const uint32_t *wp = w + (int64_t)co * wb * g.w_pitch + (r * g.S + t) * g.cw;
            for (int i = 0; i < ab; ++i)
                for (int j = 0; j < wb; ++j) {
                    int32_t x = 0;
                    for (int c = 0; c < g.cw; ++c) x += __popc(ap[i * g.a_pitch + c] ^ wp[j * g.w_pitch + c]);
                    s += x << (i + j);
                }
        }
    }
    const int32_t AB = ((1 << ab) - 1) * ((1 << wb) - 1);
    store_out(out, g.Cout, acc, m, co, g.Cout, qnn_combine(valid * g.C * AB, s), alpha);
}

// Optional fused epilogue: the next layer's encoder applied to the fp32 result.
struct NextEnc {
    uint32_t *planes;      // NULL: no encoder (then only the affine is applied)
    int bits;
    float scale;
    unsigned flags;
    const float *gamma;    // NULL: no per-feature affine
    const float *beta;
};

int check_next(const NextEnc *ne) {
    if (!ne) return QNN_OK;
    if (!ne->planes && !ne->gamma) return QNN_E_ARG;           // nothing to do beyond qnn_bgemm / qnn_bconv2d
    if (ne->beta && !ne->gamma) return QNN_E_ARG;
    if (!qnn_aligned(ne->gamma, 4) || !qnn_aligned(ne->beta, 4)) return QNN_E_ALIGN;
    if (!ne->planes) return QNN_OK;
    if (!qnn_bits_ok(ne->bits) || (ne->flags & ~QNN_RELU)) return QNN_E_ARG;
    if (!(ne->scale >= 1e-30f) || !(ne->scale <= 1e30f)) return QNN_E_SCALE;
    if (!qnn_aligned(ne->planes, 16)) return QNN_E_ALIGN;
    return QNN_OK;
}

void fill_next(qnn_tiled::Params &p, const NextEnc *ne, int Ng) {
    if (!ne) return;
    p.ch_gamma = ne->gamma;
    p.ch_beta = ne->beta;
    if (!ne->planes) return;
    p.next_planes = ne->planes;
    p.next_bits = ne->bits;
    p.next_kw = (int)qnn_row_words_i(Ng);
    p.next_inv2s = 1.0f / (2.0f * ne->scale);
    p.next_half = (float)(1 << (ne->bits - 1));
    qnn_clamp_bounds(ne->bits, ne->scale, (ne->flags & QNN_RELU) != 0, &p.next_lo, &p.next_hi);
}

void fill_next(qnn_pointwise::Params &p, const NextEnc *ne, int Ng) {
    if (!ne) return;
    p.ch_gamma = ne->gamma;
    p.ch_beta = ne->beta;
    if (!ne->planes) return;
    p.next_planes = ne->planes;
    p.next_bits = ne->bits;
    p.next_kw = (int)qnn_row_words_i(Ng);
    p.next_inv2s = 1.0f / (2.0f * ne->scale);
    p.next_half = (float)(1 << (ne->bits - 1));
    qnn_clamp_bounds(ne->bits, ne->scale, (ne->flags & QNN_RELU) != 0, &p.next_lo, &p.next_hi);
}

int bgemm_impl(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg, float alpha,
               float *out, int64_t ldo, int32_t *acc, const NextEnc *ne, void *stream);
int bconv_impl(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C, int Cout,
               int R, int S, int stride, int pad, int dil, int transposed, int out_pad, float alpha, float *out,
               int32_t *acc, const NextEnc *ne, void *stream);

}  // namespace

extern "C" int qnn_bgemm(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg,
                         float alpha, float *out, int64_t ldo, int32_t *acc, void *stream) {
    return bgemm_impl(a_planes, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, acc, nullptr, stream);
}

extern "C" int qnn_bconv2d(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C,
                           int Cout, int R, int S, int stride, int pad, float alpha, float *out, int32_t *acc,
                           void *stream) {
    return bconv_impl(a_planes, ab, w_packed, wb, N, H, W, C, Cout, R, S, stride, pad, 1, 0, 0, alpha, out, acc, nullptr,
                      stream);
}

extern "C" int qnn_bconv2d_general(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W,
                                   int C, int Cout, int R, int S, int stride, int pad, int dilation, int transposed,
                                   int out_pad, float alpha, float *out, int32_t *acc, void *stream) {
    return bconv_impl(a_planes, ab, w_packed, wb, N, H, W, C, Cout, R, S, stride, pad, dilation, transposed ? 1 : 0, out_pad,
                      alpha, out, acc, nullptr, stream);
}

extern "C" int qnn_bgemm_encode(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng,
                                int Kg, float alpha, const float *ch_gamma, const float *ch_beta, int next_bits,
                                float next_scale, unsigned next_flags, uint32_t *next_planes, float *out, int64_t ldo,
                                void *stream) {
    const NextEnc ne = {next_planes, next_bits, next_scale, next_flags, ch_gamma, ch_beta};
    return bgemm_impl(a_planes, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, nullptr, &ne, stream);
}

extern "C" int qnn_bconv2d_encode(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W,
                                  int C, int Cout, int R, int S, int stride, int pad, float alpha, const float *ch_gamma,
                                  const float *ch_beta, int next_bits, float next_scale, unsigned next_flags,
                                  uint32_t *next_planes, float *out, void *stream) {
    const NextEnc ne = {next_planes, next_bits, next_scale, next_flags, ch_gamma, ch_beta};
    return bconv_impl(a_planes, ab, w_packed, wb, N, H, W, C, Cout, R, S, stride, pad, 1, 0, 0, alpha, out, nullptr, &ne,
                      stream);
}

namespace {

// Argument checks shared by qnn_bgemm, the chaining form and the composite entry points; `has_next` = the chaining
// epilogue supplies an output of its own (next-layer planes), so out and acc may both be absent.
int bgemm_check(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg, float alpha,
                const float *out, int64_t ldo, const int32_t *acc, bool has_next) {
    if (!a_planes || !w_packed || Mg <= 0 || Ng <= 0 || Kg <= 0) return QNN_E_ARG;
    if (!out && !acc && !has_next) return QNN_E_ARG;
    if (!qnn_bits_ok(ab) || !qnn_bits_ok(wb) || (out && ldo < Ng)) return QNN_E_ARG;
    if (!isfinite(alpha)) return QNN_E_SCALE;
    if (!qnn_aligned(a_planes, 16) || !qnn_aligned(w_packed, 16) || !qnn_aligned(out, 4) || !qnn_aligned(acc, 4))
        return QNN_E_ALIGN;
    const int64_t AB = (int64_t)((1 << ab) - 1) * ((1 << wb) - 1);
    if ((int64_t)Kg * AB >= ((int64_t)1 << 31)) return QNN_E_RANGE;
    if (Mg > ((int64_t)1 << 31) - 1) return QNN_E_RANGE;
    return QNN_OK;
}

int bgemm_impl(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg, float alpha,
               float *out, int64_t ldo, int32_t *acc, const NextEnc *ne, void *stream) {
    if (!a_planes || !w_packed || Mg <= 0 || Ng <= 0 || Kg <= 0) return QNN_E_ARG;
    if (const int rc = check_next(ne)) return rc;
    if (const int rc = bgemm_check(a_planes, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, acc, ne && ne->planes)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int kw = (int)qnn_row_words_i(Kg);
    const uint32_t *w = static_cast<const uint32_t *>(w_packed);
    if (qnn_pointwise::applicable(ab, wb, Kg, Ng)) {                 // rows of at most four words per plane
        qnn_pointwise::Params d = {};
        d.a = a_planes; d.w = w; d.Mg = Mg; d.Ng = Ng; d.Kg = Kg; d.a_pitch = kw; d.w_pitch = kw;
        d.alpha = alpha; d.out = out; d.ldo = ldo; d.acc = acc; d.conv = 0;
        fill_next(d, ne, Ng);
        return qnn_pointwise::dispatch(ab, wb, d, st);
    }
    qnn_tiled::Params p = {};
    p.a = a_planes; p.w = w; p.tapsum = nullptr;
    p.Mg = Mg; p.Ng = Ng;
    p.a_pitch = kw; p.w_pitch = kw; p.kwords = kw;
    p.n_elems = Kg; p.alpha = alpha; p.out = out; p.ldo = ldo; p.acc = acc;
    fill_next(p, ne, Ng);
    return qnn_tiled::dispatch_tiled(0, ab, wb, p, st);
}

int bconv_impl(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C, int Cout,
               int R, int S, int stride, int pad, int dil, int transposed, int out_pad, float alpha, float *out,
               int32_t *acc, const NextEnc *ne, void *stream) {
    if (!a_planes || !w_packed) return QNN_E_ARG;
    if (const int rc = check_next(ne)) return rc;
    if (!out && !acc && !(ne && ne->planes)) return QNN_E_ARG;
    if (N <= 0 || H <= 0 || W <= 0 || C <= 0 || Cout <= 0 || R <= 0 || S <= 0 || stride <= 0 || pad < 0) return QNN_E_ARG;
    if (dil < 1 || out_pad < 0 || (!transposed && out_pad != 0) || (transposed && out_pad >= stride && out_pad >= dil))
        return QNN_E_ARG;
    if (!qnn_bits_ok(ab) || !qnn_bits_ok(wb)) return QNN_E_ARG;
    if (!isfinite(alpha)) return QNN_E_SCALE;
    if (!qnn_aligned(a_planes, 16) || !qnn_aligned(w_packed, 16) || !qnn_aligned(out, 4) || !qnn_aligned(acc, 4))
        return QNN_E_ALIGN;
    ConvGeom g;
    g.N = N; g.H = H; g.W = W; g.C = C; g.Cout = Cout; g.R = R; g.S = S; g.stride = stride; g.pad = pad;
    const int64_t ext_r = (int64_t)dil * (R - 1) + 1, ext_s = (int64_t)dil * (S - 1) + 1;   // extent of the dilated kernel
    int64_t ho64, wo64;
    if (!transposed) {
        if (H + 2 * (int64_t)pad < ext_r || W + 2 * (int64_t)pad < ext_s) return QNN_E_ARG;
        ho64 = (H + 2 * (int64_t)pad - ext_r) / stride + 1;
        wo64 = (W + 2 * (int64_t)pad - ext_s) / stride + 1;
    } else {
        ho64 = ((int64_t)H - 1) * stride - 2 * (int64_t)pad + ext_r + out_pad;
        wo64 = ((int64_t)W - 1) * stride - 2 * (int64_t)pad + ext_s + out_pad;
    }
    if (ho64 <= 0 || wo64 <= 0 || ho64 > 0x7fffffff || wo64 > 0x7fffffff) return QNN_E_ARG;
    g.Ho = (int)ho64;
    g.Wo = (int)wo64;
    g.cw = (C + 31) / 32;
    g.a_pitch = (int)qnn_row_words_i(C);
    g.w_pitch = (int)qnn_w_row_words_i(R * S, C);
    const int64_t AB = (int64_t)((1 << ab) - 1) * ((1 << wb) - 1);
    if ((int64_t)R * S * C * AB >= ((int64_t)1 << 31)) return QNN_E_RANGE;
    const int64_t Mg = (int64_t)N * g.Ho * g.Wo;
    if (Mg > ((int64_t)1 << 31) - 1 || (int64_t)N * H * W > ((int64_t)1 << 31) - 1) return QNN_E_RANGE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const uint32_t *w = static_cast<const uint32_t *>(w_packed);
    if (dil == 1 && !transposed && R == 1 && S == 1 && pad == 0 && C >= 32 && qnn_pointwise::applicable(ab, wb, C, Cout)) {
        // 1x1 convolution on at most 128 channels (a residual network's projections): no border, whole reduction in registers
        qnn_pointwise::Params d = {};
        d.a = a_planes; d.w = w; d.Mg = Mg; d.Ng = Cout; d.Kg = C; d.a_pitch = g.a_pitch; d.w_pitch = g.w_pitch;
        d.alpha = alpha; d.out = out; d.ldo = Cout; d.acc = acc;
        d.conv = 1; d.H = H; d.W = W; d.Ho = g.Ho; d.Wo = g.Wo; d.stride = stride;
        fill_next(d, ne, Cout);
        return qnn_pointwise::dispatch(ab, wb, d, st);
    }
    if (dil == 1 && !transposed && qnn_dense::dense1_applicable(ab, wb, R, S, C, Cout)) {
        qnn_dense::Params d = {};
        d.a = a_planes; d.w = w;
        d.tapsum = reinterpret_cast<const int32_t *>(w + (int64_t)Cout * wb * g.w_pitch);
        d.Mg = Mg; d.Ng = Cout; d.a_pitch = g.a_pitch; d.w_pitch = g.w_pitch;
        d.alpha = alpha; d.out = out; d.acc = acc;
        d.H = H; d.W = W; d.C = C; d.R = R; d.S = S; d.stride = stride; d.pad = pad; d.Ho = g.Ho; d.Wo = g.Wo;
        if (ne && !out) return QNN_E_ARG;          // this path encodes from the fp32 result in a second launch
        if (ne) { d.ch_gamma = ne->gamma; d.ch_beta = ne->beta; }
        const int rc = qnn_dense::dispatch_dense1(ab, wb, d, st);
        if (rc != QNN_OK || !ne || !ne->planes) return rc;
        return qnn_encode_pack(out, Mg, Cout, Cout, ne->bits, ne->scale, ne->flags, ne->planes, nullptr, stream);
    }
    // the tiled kernel divides by cw and S with a 20-bit multiply-shift: exact while kwords*cw and taps*S < 2^20
    if ((int64_t)R * S * g.cw * g.cw < (1 << 20) && (int64_t)R * S * S < (1 << 20) &&
        (int64_t)R * S * g.cw < 4096) {
        qnn_tiled::Params p = {};
        p.a = a_planes; p.w = w;
        p.tapsum = reinterpret_cast<const int32_t *>(w + (int64_t)Cout * wb * g.w_pitch);
        p.Mg = Mg; p.Ng = Cout;
        p.a_pitch = g.a_pitch; p.w_pitch = g.w_pitch; p.kwords = R * S * g.cw;
        p.cw_magic = (1u << 20) / (uint32_t)g.cw + 1u;
        p.s_magic = (1u << 20) / (uint32_t)S + 1u;
        p.n_elems = R * S * C; p.alpha = alpha; p.out = out; p.ldo = Cout; p.acc = acc;
        p.H = H; p.W = W; p.C = C; p.R = R; p.S = S; p.stride = stride; p.pad = pad; p.Ho = g.Ho; p.Wo = g.Wo;
        p.cw = g.cw; p.piece = (g.cw % 4 == 0) ? 4 : ((g.cw % 2 == 0) ? 2 : 1);
        p.dil = dil; p.transposed = transposed;
        fill_next(p, ne, Cout);
        int kind = (dil != 1 || transposed) ? 2 : 1;
        // nine taps and at most 4 channel words: 9-word groups leave no reduction tail (9% faster at C = 64, 128);
        // for more channels the tail is negligible and the 16-byte copies of the 8-word path win
        if (kind == 1 && R == 3 && S == 3 && g.cw <= 4 && ab <= 4 && wb <= 4) kind = 3;
        return qnn_tiled::dispatch_tiled(kind, ab, wb, p, st);
    }
    if (dil != 1 || transposed) return QNN_E_RANGE;      // the fallback kernel knows plain convolutions only
    dim3 grid((unsigned)qnn_ceil_div(Cout, 16), (unsigned)qnn_ceil_div(Mg, 16));
    if (grid.y > 65535) return QNN_E_RANGE;
    if (ne && (!out || ne->gamma)) return QNN_E_ARG;   // the fallback kernel has no affine epilogue
    bconv_generic_kernel<<<grid, 256, 0, st>>>(a_planes, ab, w, wb, g, alpha, out, acc);
    if (cudaGetLastError() != cudaSuccess) return QNN_E_CUDA;
    if (!ne || !ne->planes) return QNN_OK;
    return qnn_encode_pack(out, Mg, Cout, Cout, ne->bits, ne->scale, ne->flags, ne->planes, nullptr, stream);
}

}  // namespace

// Popcount instructions per output (all plane pairs) of the kernel that bgemm_impl / bconv_impl pick for a layer
// (plain convolution: dilation 1, not transposed); mirrors their dispatch.
extern "C" int64_t qnn_popcounts_per_output(int ab, int wb, int is_conv, int R, int S, int C, int Cout) {
    if (!qnn_bits_ok(ab) || !qnn_bits_ok(wb) || R < 1 || S < 1 || C < 1 || Cout < 1 || (!is_conv && R * S != 1)) return 0;
    const int64_t cw = (C + 31) / 32, pairs = (int64_t)ab * wb;
    if ((!is_conv || (R == 1 && S == 1 && C >= 32)) && qnn_pointwise::applicable(ab, wb, C, Cout))
        return qnn_pointwise::weighted_count_popcounts(ab, wb, (int)cw);          // (1x1 convolutions: when pad = 0)
    if (is_conv && qnn_dense::dense1_applicable(ab, wb, R, S, C, Cout))
        return (ab == 4 && wb == 4) ? 10 : ((ab == 3 && wb == 3) ? 7 : pairs);
    if (is_conv && R == 3 && S == 3 && cw <= 4 && ab <= 4 && wb <= 4) return pairs * cw * 4;    // 9-word groups
    qnn_tiled::Params p = {};
    p.kwords = is_conv ? (int)(R * S * cw) : (int)qnn_row_words_i(C);
    qnn_tiled::set_k_split(p);
    return pairs * ((int64_t)p.nfull * 4 + p.ntail);
}

int qnn_check_bgemm(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg, float alpha,
                    const float *out, int64_t ldo, const int32_t *acc) {
    return bgemm_check(a_planes, ab, w_packed, wb, Mg, Ng, Kg, alpha, out, ldo, acc, false);
}

extern "C" int qnn_fc_forward_host(const float *x_host, int64_t Mg, int Kg, int ab, float scale_a, unsigned flags,
                                   const void *w_packed, int wb, int Ng, float alpha, float *out_host, float *x_dev,
                                   uint32_t *planes_dev, float *out_dev, void *stream) {
    if (!x_host || !out_host || !x_dev || !planes_dev || !out_dev || Mg <= 0 || Kg <= 0 || Ng <= 0) return QNN_E_ARG;
    // every argument error of the two kernels is found here, before the first copy is enqueued
    if (const int rc = qnn_check_encode_pack(x_dev, Mg, Kg, Kg, ab, scale_a, flags, planes_dev, nullptr)) return rc;
    if (const int rc = qnn_check_bgemm(planes_dev, ab, w_packed, wb, Mg, Ng, Kg, alpha, out_dev, Ng, nullptr)) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(x_dev, x_host, (size_t)Mg * Kg * sizeof(float), cudaMemcpyHostToDevice, st) != cudaSuccess)
        return QNN_E_CUDA;
    int rc = qnn_encode_pack(x_dev, Mg, Kg, Kg, ab, scale_a, flags, planes_dev, nullptr, stream);
    if (rc != QNN_OK) return rc;
    rc = qnn_bgemm(planes_dev, ab, w_packed, wb, Mg, Ng, Kg, alpha, out_dev, Ng, nullptr, stream);
    if (rc != QNN_OK) return rc;
    if (cudaMemcpyAsync(out_host, out_dev, (size_t)Mg * Ng * sizeof(float), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return QNN_E_CUDA;
    return QNN_OK;
}

extern "C" int qnn_fc_forward_host_pipelined(const float *x_host, int64_t Mg, int Kg, int ab, float scale_a,
                                             unsigned flags, const void *w_packed, int wb, int Ng, float alpha,
                                             float *out_host, float *x_dev, uint32_t *planes_dev, float *out_dev,
                                             int64_t rows_per_chunk, void *const *streams, int nstreams) {
    if (!x_host || !out_host || !x_dev || !planes_dev || !out_dev || !streams || Mg <= 0 || Kg <= 0 || Ng <= 0)
        return QNN_E_ARG;
    if (nstreams < 1 || rows_per_chunk < 1 || !qnn_bits_ok(ab)) return QNN_E_ARG;
    // Every argument error of the two kernels is found here, before the first chunk is enqueued: a chunk is a row
    // range of the same buffers (rows of planes are multiples of 16 bytes), so it passes whatever the whole passes.
    if (const int rc = qnn_check_encode_pack(x_dev, Mg, Kg, Kg, ab, scale_a, flags, planes_dev, nullptr)) return rc;
    if (const int rc = qnn_check_bgemm(planes_dev, ab, w_packed, wb, Mg, Ng, Kg, alpha, out_dev, Ng, nullptr)) return rc;
    const int64_t plane_words_per_row = (int64_t)ab * qnn_row_words_i(Kg);
    int64_t chunk = 0;
    for (int64_t r0 = 0; r0 < Mg; r0 += rows_per_chunk, ++chunk) {
        const int64_t rows = (Mg - r0 < rows_per_chunk) ? (Mg - r0) : rows_per_chunk;
        void *stream = streams[chunk % nstreams];
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        float *xd = x_dev + r0 * Kg;
        uint32_t *pd = planes_dev + r0 * plane_words_per_row;
        float *od = out_dev + r0 * Ng;
        if (cudaMemcpyAsync(xd, x_host + r0 * Kg, (size_t)rows * Kg * sizeof(float), cudaMemcpyHostToDevice, st) !=
            cudaSuccess)
            return QNN_E_CUDA;
        int rc = qnn_encode_pack(xd, rows, Kg, Kg, ab, scale_a, flags, pd, nullptr, stream);
        if (rc != QNN_OK) return rc;
        rc = qnn_bgemm(pd, ab, w_packed, wb, rows, Ng, Kg, alpha, od, Ng, nullptr, stream);
        if (rc != QNN_OK) return rc;
        if (cudaMemcpyAsync(out_host + r0 * Ng, od, (size_t)rows * Ng * sizeof(float), cudaMemcpyDeviceToHost, st) !=
            cudaSuccess)
            return QNN_E_CUDA;
    }
    return QNN_OK;
}

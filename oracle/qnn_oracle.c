/*
 * qnn_oracle.c -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of what one {-1,+1}-decomposed
 * quantized layer computes.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library never does, and the
 * two share no source, header, table or helper.
 *
 * The paper's multi-branch product (Eq. 8) is an identity, not an approximation:
 * the weighted sum of all plane-pair xnor/popcount products equals the ordinary
 * integer dot product of the odd-integer codes.  The oracle is therefore the
 * plain definition:
 *
 *   1. quantize each real tensor to odd codes q in {-(2^b-1), ..., -1, +1, ...,
 *      2^b-1} (code space of Eq. 7 / Section 3.2; interval ownership of Table 2),
 *   2. naive integer matrix product / zero-padded convolution of the codes
 *      (Eq. 1 applied to codes; Op(EnC(x), EnC(w)) of Eq. 9),
 *   3. one multiplication by the layer scale (Eq. 9, Alg. 1 forward step
 *      "a_l <- r * a_hat / ((2^M-1)(2^K-1))").
 *
 * It also writes the canonical bit-plane storage (Eq. 3 / Eq. 7: plane m holds
 * c_m of every element, one bit per element, +1 stored as 1) so that packed
 * planes can be compared word for word, and states Eq. 8 itself on those
 * planes (oracle_fc_bitplanes: one xor and one popcount per word and plane
 * pair), which must agree exactly with the plain product of step 2.
 *
 * Floating point: the quantizer decides an integer from binary32 data, so the
 * decision is fixed to one binary32 evaluation order: v = fma(x, 1/(2s), 2^(b-1))
 * with a single rounding (Table 2's interval ends are where v is an integer);
 * everything after it is integer until the single binary32 multiply of step 3.
 *
 * Parallelism: independent output rows are spread over OpenMP threads.  There is
 * no blocking, vectorisation by hand, fusion or reordering.
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_E_ARG (-1)
#define ORACLE_E_RANGE (-3)

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/*
 * Quantizer (Table 2 generalised to b bits; code space of Section 3.2).
 * scale = s = r / (2^b - 1) is the distance from 0 to the first grid point; grid
 * points are q*s for odd q.  Interval ownership follows Table 2: a value exactly
 * half-way between two grid points goes to the one farther from zero, and 0
 * itself belongs to the negative side ("(-2/3, 0]" maps to -1/3).
 * Values outside [-r, r] take the end codes (the clamp of Eq. 15).
 * Returns the unsigned code t in [0, 2^b - 1]; the odd code is q = 2t - (2^b-1).
 */
static int quantize_t(float x, float inv2s, int bits, int relu) {
    const float amax = (float)((1 << bits) - 1);
    const float half = (float)(1 << (bits - 1));
    if (relu) x = fmaxf(x, 0.0f);
    float v = fmaf(x, inv2s, half);              /* x/(2s) + 2^(b-1), one rounding */
    float tf = (x > 0.0f) ? floorf(v) : ceilf(v) - 1.0f;
    tf = fminf(fmaxf(tf, 0.0f), amax);           /* end codes; NaN -> 0 */
    return (int)tf;
}

/* x[n] -> odd codes q[n].  relu != 0 applies max(x,0) first. */
int oracle_quantize(const float *x, size_t n, int bits, float scale, int relu, int16_t *q) {
    if (!x || !q || bits < 1 || bits > 8) return ORACLE_E_ARG;
    if (!(scale > 0.0f) || isinf(scale)) return ORACLE_E_ARG;
    const float inv2s = 1.0f / (2.0f * scale);
    const int amax = (1 << bits) - 1;
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i) {
        int t = quantize_t(x[i], inv2s, bits, relu);
        q[i] = (int16_t)(2 * t - amax);
    }
    return ORACLE_OK;
}

/* Number of 32-bit words one plane of one row occupies: ceil(k/32) rounded up to 4. */
size_t oracle_row_words(size_t k) {
    size_t w = (k + 31) / 32;
    return (w + 3) / 4 * 4;
}

/*
 * Canonical bit planes of odd codes (Eq. 7: q = sum_m 2^(m-1) c_m, c_m = +-1).
 * With t = (q + 2^b - 1)/2, c_m = +1 exactly when binary bit (m-1) of t is 1.
 * Layout: planes[row][plane i = m-1][word], element k in bit (k mod 32) of word
 * (k div 32); all padding bits are 0.
 */
int oracle_pack_planes(const int16_t *q, size_t rows, size_t k, int bits, uint32_t *planes) {
    if (!q || !planes || bits < 1 || bits > 8) return ORACLE_E_ARG;
    const size_t kw = oracle_row_words(k);
    const int amax = (1 << bits) - 1;
#pragma omp parallel for schedule(static)
    for (ptrdiff_t r = 0; r < (ptrdiff_t)rows; ++r) {
        for (int i = 0; i < bits; ++i) {
            uint32_t *dst = planes + ((size_t)r * bits + i) * kw;
            for (size_t w = 0; w < kw; ++w) dst[w] = 0u;
            for (size_t e = 0; e < k; ++e) {
                int t = (q[(size_t)r * k + e] + amax) / 2;
                if ((t >> i) & 1) dst[e / 32] |= (uint32_t)1 << (e % 32);
            }
        }
    }
    return ORACLE_OK;
}

/* acc[m][n] = sum_k qa[m][k] * qw[n][k]   (fully-connected layer on codes). */
int oracle_fc(const int16_t *qa, const int16_t *qw, size_t Mg, size_t Ng, size_t Kg, int32_t *acc) {
    if (!qa || !qw || !acc) return ORACLE_E_ARG;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (ptrdiff_t m = 0; m < (ptrdiff_t)Mg; ++m) {
        for (size_t n = 0; n < Ng; ++n) {
            int64_t s = 0;
            for (size_t k = 0; k < Kg; ++k)
                s += (int64_t)qa[(size_t)m * Kg + k] * (int64_t)qw[n * Kg + k];
            if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
            acc[(size_t)m * Ng + n] = (int32_t)s;
        }
    }
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/* Eq. 8 written out on the packed planes (the decomposition itself, not its result's plain definition):
 * acc[m][n] = sum_i sum_j 2^(i+j) * (Kg - 2 * popcount(a_i[m] xor w_j[n])), planes as oracle_pack_planes lays them out
 * ([rows][bits][words], padding bits zero in both operands, so they never differ).  One xor and one popcount per
 * 32-bit word and plane pair, nothing blocked or combined.  Serves as a second, independent statement of oracle_fc
 * (the two must agree exactly) and as the CPU form of the method that the efficiency experiment (Section 5.4) times. */
int oracle_fc_bitplanes(const uint32_t *a_planes, const uint32_t *w_planes, size_t Mg, size_t Ng, size_t Kg, int ab, int wb,
                        int32_t *acc) {
    if (!a_planes || !w_planes || !acc || ab < 1 || ab > 8 || wb < 1 || wb > 8) return ORACLE_E_ARG;
    const size_t kw = oracle_row_words(Kg);
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (ptrdiff_t m = 0; m < (ptrdiff_t)Mg; ++m) {
        for (size_t n = 0; n < Ng; ++n) {
            int64_t s = 0;
            for (int i = 0; i < ab; ++i)
                for (int j = 0; j < wb; ++j) {
                    const uint32_t *a = a_planes + ((size_t)m * ab + i) * kw;
                    const uint32_t *w = w_planes + (n * wb + j) * kw;
                    int64_t differ = 0;
                    for (size_t x = 0; x < kw; ++x) differ += __builtin_popcount(a[x] ^ w[x]);
                    s += ((int64_t)Kg - 2 * differ) * ((int64_t)1 << (i + j));
                }
            if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
            acc[(size_t)m * Ng + n] = (int32_t)s;
        }
    }
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/* The same dot product for a list of (row, column) pairs only. */
int oracle_fc_sampled(const int16_t *qa, const int16_t *qw, size_t Kg, size_t count,
                      const int64_t *rows, const int64_t *cols, int32_t *acc) {
    if (!qa || !qw || !acc || !rows || !cols) return ORACLE_E_ARG;
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)count; ++i) {
        const int16_t *a = qa + (size_t)rows[i] * Kg;
        const int16_t *w = qw + (size_t)cols[i] * Kg;
        int64_t s = 0;
        for (size_t k = 0; k < Kg; ++k) s += (int64_t)a[k] * (int64_t)w[k];
        if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
        acc[i] = (int32_t)s;
    }
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/*
 * One output of the convolution of codes.  Activations are [N][H][W][C], weights
 * [Cout][R][S][C]; the encoded tensor is padded with true zeros, so a tap that
 * falls outside the image adds nothing (0 is not a code; Eq. 9 applies the layer
 * operation to the already-encoded tensor).
 */
static int64_t conv_one(const int16_t *qa, const int16_t *qw, int H, int W, int C, int R, int S,
                        int stride, int pad, int n, int ho, int wo, int co) {
    int64_t s = 0;
    for (int r = 0; r < R; ++r) {
        int hi = ho * stride - pad + r;
        if (hi < 0 || hi >= H) continue;
        for (int t = 0; t < S; ++t) {
            int wi = wo * stride - pad + t;
            if (wi < 0 || wi >= W) continue;
            const int16_t *a = qa + (((size_t)n * H + hi) * W + wi) * C;
            const int16_t *w = qw + (((size_t)co * R + r) * S + t) * C;
            for (int c = 0; c < C; ++c) s += (int64_t)a[c] * (int64_t)w[c];
        }
    }
    return s;
}

int oracle_conv_out_dim(int in, int k, int stride, int pad) {
    return (in + 2 * pad - k) / stride + 1;
}

/* acc[n][ho][wo][co], Ho = (H + 2 pad - R)/stride + 1, Wo likewise. */
int oracle_conv2d(const int16_t *qa, const int16_t *qw, int N, int H, int W, int C, int Cout, int R,
                  int S, int stride, int pad, int32_t *acc) {
    if (!qa || !qw || !acc || stride < 1 || pad < 0) return ORACLE_E_ARG;
    const int Ho = oracle_conv_out_dim(H, R, stride, pad);
    const int Wo = oracle_conv_out_dim(W, S, stride, pad);
    if (Ho < 1 || Wo < 1) return ORACLE_E_ARG;
    int bad = 0;
    const ptrdiff_t rows = (ptrdiff_t)N * Ho * Wo;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (ptrdiff_t m = 0; m < rows; ++m) {
        int n = (int)(m / ((ptrdiff_t)Ho * Wo));
        int ho = (int)((m / Wo) % Ho);
        int wo = (int)(m % Wo);
        for (int co = 0; co < Cout; ++co) {
            int64_t s = conv_one(qa, qw, H, W, C, R, S, stride, pad, n, ho, wo, co);
            if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
            acc[(size_t)m * Cout + co] = (int32_t)s;
        }
    }
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/* Convolution outputs for a list of (output row m = (n*Ho+ho)*Wo+wo, channel co) pairs. */
int oracle_conv2d_sampled(const int16_t *qa, const int16_t *qw, int N, int H, int W, int C, int Cout,
                          int R, int S, int stride, int pad, size_t count, const int64_t *rows,
                          const int64_t *cols, int32_t *acc) {
    if (!qa || !qw || !acc || !rows || !cols || stride < 1 || pad < 0) return ORACLE_E_ARG;
    (void)N; (void)Cout;
    const int Ho = oracle_conv_out_dim(H, R, stride, pad);
    const int Wo = oracle_conv_out_dim(W, S, stride, pad);
    int bad = 0;
#pragma omp parallel for schedule(static) reduction(| : bad)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)count; ++i) {
        int64_t m = rows[i];
        int n = (int)(m / ((int64_t)Ho * Wo));
        int ho = (int)((m / Wo) % Ho);
        int wo = (int)(m % Wo);
        int64_t s = conv_one(qa, qw, H, W, C, R, S, stride, pad, n, ho, wo, (int)cols[i]);
        if (s > INT32_MAX || s < INT32_MIN) bad |= 1;
        acc[i] = (int32_t)s;
    }
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/* out = float(acc) * alpha: one int->binary32 conversion (round to nearest even), one multiply. */
int oracle_scale(const int32_t *acc, size_t n, float alpha, float *out) {
    if (!acc || !out) return ORACLE_E_ARG;
#pragma omp parallel for schedule(static)
    for (ptrdiff_t i = 0; i < (ptrdiff_t)n; ++i) out[i] = (float)acc[i] * alpha;
    return ORACLE_OK;
}

/*
 * Per-feature affine after the scale (a folded batch-normalisation; Section 3.2 notes that when batch
 * normalisation follows, the fixed scaling factor is dropped, i.e. alpha = 1 and the affine carries the scale):
 * y[m][n] = fma(y[m][n], gamma[n], beta[n]) in binary32, one rounding.  beta may be NULL (0).
 */
int oracle_affine(float *y, size_t rows, size_t Ng, const float *gamma, const float *beta) {
    if (!y || !gamma) return ORACLE_E_ARG;
#pragma omp parallel for schedule(static)
    for (ptrdiff_t m = 0; m < (ptrdiff_t)rows; ++m)
        for (size_t n = 0; n < Ng; ++n) y[(size_t)m * Ng + n] = fmaf(y[(size_t)m * Ng + n], gamma[n], beta ? beta[n] : 0.0f);
    return ORACLE_OK;
}

/*
 * Convolution with dilation, and transposed convolution ("deconvolution", Section 3.2), on codes.
 * Forward:     acc[n,ho,wo,co] = sum_{r,s,c} qa[n, ho*stride - pad + r*dil, wo*stride - pad + s*dil, c] * qw[co,r,s,c]
 * Transposed:  every input pixel (hi, wi) adds qa[n,hi,wi,c]*qw[co,r,s,c] to output (hi*stride - pad + r*dil,
 *              wi*stride - pad + s*dil); Ho = (H-1)*stride - 2*pad + dil*(R-1) + 1 + out_pad, Wo likewise.
 * Positions outside the tensors contribute nothing (the encoded tensor is surrounded by, and for the transposed
 * form interleaved with, true zeros).  The transposed form is written as the scatter it is defined by.
 */
int oracle_conv2d_general(const int16_t *qa, const int16_t *qw, int N, int H, int W, int C, int Cout, int R, int S,
                          int stride, int pad, int dil, int transposed, int out_pad, int32_t *acc) {
    if (!qa || !qw || !acc || stride < 1 || pad < 0 || dil < 1 || out_pad < 0) return ORACLE_E_ARG;
    int Ho, Wo;
    if (!transposed) {
        Ho = (H + 2 * pad - dil * (R - 1) - 1) / stride + 1;
        Wo = (W + 2 * pad - dil * (S - 1) - 1) / stride + 1;
    } else {
        Ho = (H - 1) * stride - 2 * pad + dil * (R - 1) + 1 + out_pad;
        Wo = (W - 1) * stride - 2 * pad + dil * (S - 1) + 1 + out_pad;
    }
    if (Ho < 1 || Wo < 1) return ORACLE_E_ARG;
    const size_t total = (size_t)N * Ho * Wo * Cout;
    int64_t *wide = (int64_t *)calloc(total, sizeof(int64_t));
    if (!wide) return ORACLE_E_ARG;
    if (!transposed) {
#pragma omp parallel for schedule(static)
        for (ptrdiff_t m = 0; m < (ptrdiff_t)N * Ho * Wo; ++m) {
            int n = (int)(m / ((ptrdiff_t)Ho * Wo)), ho = (int)((m / Wo) % Ho), wo = (int)(m % Wo);
            for (int co = 0; co < Cout; ++co) {
                int64_t sum = 0;
                for (int r = 0; r < R; ++r) {
                    int hi = ho * stride - pad + r * dil;
                    if (hi < 0 || hi >= H) continue;
                    for (int t = 0; t < S; ++t) {
                        int wi = wo * stride - pad + t * dil;
                        if (wi < 0 || wi >= W) continue;
                        const int16_t *a = qa + (((size_t)n * H + hi) * W + wi) * C;
                        const int16_t *w = qw + (((size_t)co * R + r) * S + t) * C;
                        for (int c = 0; c < C; ++c) sum += (int64_t)a[c] * (int64_t)w[c];
                    }
                }
                wide[(size_t)m * Cout + co] = sum;
            }
        }
    } else {
#pragma omp parallel for schedule(static)
        for (ptrdiff_t n = 0; n < N; ++n)           /* images are independent; the scatter inside one is serial */
            for (int hi = 0; hi < H; ++hi)
                for (int wi = 0; wi < W; ++wi) {
                    const int16_t *a = qa + (((size_t)n * H + hi) * W + wi) * C;
                    for (int r = 0; r < R; ++r) {
                        int ho = hi * stride - pad + r * dil;
                        if (ho < 0 || ho >= Ho) continue;
                        for (int t = 0; t < S; ++t) {
                            int wo = wi * stride - pad + t * dil;
                            if (wo < 0 || wo >= Wo) continue;
                            for (int co = 0; co < Cout; ++co) {
                                const int16_t *w = qw + (((size_t)co * R + r) * S + t) * C;
                                int64_t sum = 0;
                                for (int c = 0; c < C; ++c) sum += (int64_t)a[c] * (int64_t)w[c];
                                wide[(((size_t)n * Ho + ho) * Wo + wo) * Cout + co] += sum;
                            }
                        }
                    }
                }
    }
    int bad = 0;
    for (size_t i = 0; i < total; ++i) {
        if (wide[i] > INT32_MAX || wide[i] < INT32_MIN) bad = 1;
        acc[i] = (int32_t)wide[i];
    }
    free(wide);
    return bad ? ORACLE_E_RANGE : ORACLE_OK;
}

/*
 * Trigonometric M-bit encoder (Eq. 10) and its straight-through derivative (Eq. 12), the training-side form of
 * the encoder.  With xn = x / r and k_m = (2^M - 1) / 2^m:
 *   phi_M^M(xn) = sign(sin(k_M pi xn)),   phi_M^m(xn) = sign(-sin(k_m pi xn)) for m < M,
 *   d phi_M^m / d xn = +- k_m pi cos(k_m pi xn) for |xn| <= 1, else 0 (sign + for m = M, - otherwise).
 * Forward: the sign is a decision on binary32 data, and Eq. 10 does not say in which precision its argument is
 * formed.  Reading taken: xn = x / r and y = k_m * xn are one binary32 division and one binary32 product (k_m
 * is exactly representable); sign(sin(pi y)) is then decided exactly from y: 0 when y is an integer, positive
 * when floor(y) is even and negative when it is odd -- no library sine is involved, so the decision is
 * reproducible and matches the exact sign of the sine of pi * y.
 * c[(m-1)*n + e] receives phi_M^m of element e as -1, 0 or +1.
 */
int oracle_mbit_encoder_forward(const float *x, size_t n, int bits, float r, float *c) {
    if (!x || !c || bits < 1 || bits > 8 || !(r > 0.0f)) return ORACLE_E_ARG;
    for (int m = 1; m <= bits; ++m) {
        const float k = (float)((1 << bits) - 1) / (float)(1 << m);
        for (size_t e = 0; e < n; ++e) {
            const float xn = x[e] / r;
            const float y = k * xn;
            const float fl = floorf(y);
            float sgn;
            if (!(y == y) || isinf(y)) sgn = 0.0f;                    /* NaN / infinity: no state */
            else if (fl == y) sgn = 0.0f;
            else sgn = (fmodf(fl, 2.0f) == 0.0f) ? 1.0f : -1.0f;       /* sin(pi y) > 0 on (2j, 2j+1) */
            c[(size_t)(m - 1) * n + e] = (m == bits) ? sgn : -sgn;
        }
    }
    return ORACLE_OK;
}

/* gx[e] = (1/r) * sum_m gc[m-1][e] * d phi_M^m / d xn, evaluated in binary64 (Eq. 12; zero outside [-1, 1]). */
int oracle_mbit_encoder_backward(const float *x, const float *gc, size_t n, int bits, float r, double *gx) {
    if (!x || !gc || !gx || bits < 1 || bits > 8 || !(r > 0.0f)) return ORACLE_E_ARG;
    const double pi = 3.14159265358979323846;
    for (size_t e = 0; e < n; ++e) {
        const double xn = (double)(x[e] / r);                          /* xn as Eq. 10 forms it: one binary32 division */
        double g = 0.0;
        if (xn >= -1.0 && xn <= 1.0) {
            for (int m = 1; m <= bits; ++m) {
                const double k = (double)((1 << bits) - 1) / (double)(1 << m);
                const double d = k * pi * cos(k * pi * xn);
                g += (double)gc[(size_t)(m - 1) * n + e] * ((m == bits) ? d : -d);
            }
        }
        gx[e] = g / (double)r;
    }
    return ORACLE_OK;
}

/*
 * Backward products of one fully-connected layer (Algorithm 1, backward propagation).
 * Forward (Algorithm 1, forward propagation): a_hat[r][n] = sum_m sum_j 2^(m+j-2) sum_k a^m[r][k] * W^j[n][k] and
 * a = alpha * a_hat, with a^m, W^j in {-1,+1} the planes of the odd codes qa (ab planes) and qw (wb planes):
 * q = sum_i 2^(i-1) * plane_i(q).  Given g = dC/da (binary32 input, all arithmetic here in binary64):
 *   g_hat            = alpha * g
 *   g_a^m [r][k]     = sum_j 2^(m+j-2) * sum_n g_hat[r][n] * W^j[n][k]        m = 1..ab
 *   g_W^j [n][k]     = sum_m 2^(m+j-2) * sum_r g_hat[r][n] * a^m[r][k]        j = 1..wb
 * The loops follow the algorithm's order (planes outside, contraction inside); no regrouping into codes.
 */
static double plane_of(int q, int bits, int i) {                      /* i = 1..bits; q odd in [-(2^bits-1), 2^bits-1] */
    const int t = (q + ((1 << bits) - 1)) / 2;
    return ((t >> (i - 1)) & 1) ? 1.0 : -1.0;
}

static int codes_ok(const int16_t *q, size_t n, int bits) {
    const int A = (1 << bits) - 1;
    for (size_t i = 0; i < n; ++i)
        if (q[i] < -A || q[i] > A || ((q[i] & 1) == 0)) return 0;
    return 1;
}

/* ga[(m-1)*Mg*Kg + r*Kg + k] = g_a^m[r][k] */
int oracle_fc_backward_data(const float *g, const int16_t *qw, size_t Mg, size_t Ng, size_t Kg, int ab, int wb,
                            float alpha, double *ga) {
    if (!g || !qw || !ga || ab < 1 || ab > 8 || wb < 1 || wb > 8) return ORACLE_E_ARG;
    if (!codes_ok(qw, Ng * Kg, wb)) return ORACLE_E_ARG;
    for (int m = 1; m <= ab; ++m) {
#pragma omp parallel for schedule(static)
        for (size_t r = 0; r < Mg; ++r)
            for (size_t k = 0; k < Kg; ++k) {
                double sum = 0.0;
                for (int j = 1; j <= wb; ++j) {
                    double part = 0.0;
                    for (size_t n = 0; n < Ng; ++n)
                        part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qw[n * Kg + k], wb, j);
                    sum += ldexp(part, m + j - 2);
                }
                ga[((size_t)(m - 1) * Mg + r) * Kg + k] = sum;
            }
    }
    return ORACLE_OK;
}

/* gw[(j-1)*Ng*Kg + n*Kg + k] = g_W^j[n][k] */
int oracle_fc_backward_weights(const float *g, const int16_t *qa, size_t Mg, size_t Ng, size_t Kg, int ab, int wb,
                               float alpha, double *gw) {
    if (!g || !qa || !gw || ab < 1 || ab > 8 || wb < 1 || wb > 8) return ORACLE_E_ARG;
    if (!codes_ok(qa, Mg * Kg, ab)) return ORACLE_E_ARG;
    for (int j = 1; j <= wb; ++j) {
#pragma omp parallel for schedule(static)
        for (size_t n = 0; n < Ng; ++n)
            for (size_t k = 0; k < Kg; ++k) {
                double sum = 0.0;
                for (int m = 1; m <= ab; ++m) {
                    double part = 0.0;
                    for (size_t r = 0; r < Mg; ++r)
                        part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qa[r * Kg + k], ab, m);
                    sum += ldexp(part, m + j - 2);
                }
                gw[((size_t)(j - 1) * Ng + n) * Kg + k] = sum;
            }
    }
    return ORACLE_OK;
}

/* The same two gradients at `count` sampled positions only (for sizes where the full loops take too long):
 * out[(p-1)*count + i] = g_a^p[rows[i]][cols[i]]  resp.  g_W^p[rows[i]][cols[i]]. */
int oracle_fc_backward_data_sampled(const float *g, const int16_t *qw, size_t Ng, size_t Kg, int ab, int wb, float alpha,
                                    size_t count, const int64_t *rows, const int64_t *cols, double *out) {
    if (!g || !qw || !out || !rows || !cols || ab < 1 || ab > 8 || wb < 1 || wb > 8) return ORACLE_E_ARG;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < count; ++i) {
        const size_t r = (size_t)rows[i], k = (size_t)cols[i];
        for (int m = 1; m <= ab; ++m) {
            double sum = 0.0;
            for (int j = 1; j <= wb; ++j) {
                double part = 0.0;
                for (size_t n = 0; n < Ng; ++n)
                    part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qw[n * Kg + k], wb, j);
                sum += ldexp(part, m + j - 2);
            }
            out[(size_t)(m - 1) * count + i] = sum;
        }
    }
    return ORACLE_OK;
}

int oracle_fc_backward_weights_sampled(const float *g, const int16_t *qa, size_t Mg, size_t Ng, size_t Kg, int ab, int wb,
                                       float alpha, size_t count, const int64_t *rows, const int64_t *cols, double *out) {
    if (!g || !qa || !out || !rows || !cols || ab < 1 || ab > 8 || wb < 1 || wb > 8) return ORACLE_E_ARG;
#pragma omp parallel for schedule(static)
    for (size_t i = 0; i < count; ++i) {
        const size_t n = (size_t)rows[i], k = (size_t)cols[i];
        for (int j = 1; j <= wb; ++j) {
            double sum = 0.0;
            for (int m = 1; m <= ab; ++m) {
                double part = 0.0;
                for (size_t r = 0; r < Mg; ++r)
                    part += ((double)alpha * (double)g[r * Ng + n]) * plane_of(qa[r * Kg + k], ab, m);
                sum += ldexp(part, m + j - 2);
            }
            out[(size_t)(j - 1) * count + i] = sum;
        }
    }
    return ORACLE_OK;
}

/* ---- Backward products of a convolution layer (Algorithm 1, backward propagation, with forward() a convolution).
 * Forward: out[n][ho][wo][co] = alpha * sum_m sum_j 2^(m+j-2) * sum_{r,s,c} a^m[n][ho*st-pad+r][wo*st-pad+s][c] * W^j[co][r][s][c],
 * taps outside the image contributing nothing.  Each gradient is the derivative of that expression, written as the
 * scatter / correlation it defines; g = dC/d(out), fp32 [N][Ho][Wo][Cout]. */

/* ga[(m-1)*N*H*W*C + ((n*H + h)*W + w)*C + c] = g_{a^m}[n][h][w][c]: every (output, tap) that read the element
 * sends its share back to it. */
int oracle_conv_backward_data(const float *g, const int16_t *qw, int N, int H, int W, int C, int Cout, int R, int S,
                              int stride, int pad, int ab, int wb, float alpha, double *ga) {
    if (!g || !qw || !ga || ab < 1 || ab > 8 || wb < 1 || wb > 8 || stride < 1 || pad < 0) return ORACLE_E_ARG;
    if (!codes_ok(qw, (size_t)Cout * R * S * C, wb)) return ORACLE_E_ARG;
    const int Ho = oracle_conv_out_dim(H, R, stride, pad), Wo = oracle_conv_out_dim(W, S, stride, pad);
    if (Ho < 1 || Wo < 1) return ORACLE_E_ARG;
    const size_t img = (size_t)H * W * C, all = (size_t)N * img;
    for (size_t i = 0; i < (size_t)ab * all; ++i) ga[i] = 0.0;
    for (int m = 1; m <= ab; ++m) {
#pragma omp parallel for schedule(static)
        for (int n = 0; n < N; ++n)
            for (int ho = 0; ho < Ho; ++ho)
                for (int wo = 0; wo < Wo; ++wo)
                    for (int r = 0; r < R; ++r)
                        for (int s = 0; s < S; ++s) {
                            const int hi = ho * stride - pad + r, wi = wo * stride - pad + s;
                            if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                            double *dst = ga + (size_t)(m - 1) * all + (size_t)n * img + ((size_t)hi * W + wi) * C;
                            const float *gp = g + (((size_t)n * Ho + ho) * Wo + wo) * Cout;
                            for (int c = 0; c < C; ++c) {
                                double sum = 0.0;
                                for (int j = 1; j <= wb; ++j) {
                                    double part = 0.0;
                                    for (int co = 0; co < Cout; ++co)
                                        part += ((double)alpha * (double)gp[co]) *
                                                plane_of(qw[(((size_t)co * R + r) * S + s) * C + c], wb, j);
                                    sum += ldexp(part, m + j - 2);
                                }
                                dst[c] += sum;
                            }
                        }
    }
    return ORACLE_OK;
}

/* gw[(j-1)*Cout*R*S*C + ((co*R + r)*S + s)*C + c] = g_{W^j}[co][r][s][c]: correlation of g with the activation planes. */
int oracle_conv_backward_weights(const float *g, const int16_t *qa, int N, int H, int W, int C, int Cout, int R, int S,
                                 int stride, int pad, int ab, int wb, float alpha, double *gw) {
    if (!g || !qa || !gw || ab < 1 || ab > 8 || wb < 1 || wb > 8 || stride < 1 || pad < 0) return ORACLE_E_ARG;
    if (!codes_ok(qa, (size_t)N * H * W * C, ab)) return ORACLE_E_ARG;
    const int Ho = oracle_conv_out_dim(H, R, stride, pad), Wo = oracle_conv_out_dim(W, S, stride, pad);
    if (Ho < 1 || Wo < 1) return ORACLE_E_ARG;
    const size_t wsz = (size_t)Cout * R * S * C;
    for (int j = 1; j <= wb; ++j) {
#pragma omp parallel for schedule(static)
        for (int co = 0; co < Cout; ++co)
            for (int r = 0; r < R; ++r)
                for (int s = 0; s < S; ++s)
                    for (int c = 0; c < C; ++c) {
                        double sum = 0.0;
                        for (int m = 1; m <= ab; ++m) {
                            double part = 0.0;
                            for (int n = 0; n < N; ++n)
                                for (int ho = 0; ho < Ho; ++ho)
                                    for (int wo = 0; wo < Wo; ++wo) {
                                        const int hi = ho * stride - pad + r, wi = wo * stride - pad + s;
                                        if (hi < 0 || hi >= H || wi < 0 || wi >= W) continue;
                                        part += ((double)alpha * (double)g[(((size_t)n * Ho + ho) * Wo + wo) * Cout + co]) *
                                                plane_of(qa[(((size_t)n * H + hi) * W + wi) * C + c], ab, m);
                                    }
                            sum += ldexp(part, m + j - 2);
                        }
                        gw[(size_t)(j - 1) * wsz + (((size_t)co * R + r) * S + s) * C + c] = sum;
                    }
    }
    return ORACLE_OK;
}

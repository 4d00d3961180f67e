/*
 * qnn.h -- C ABI of libqnn: one quantized layer computed through the {-1,+1}
 * bit-plane decomposition (arXiv 2106.09886), for NVIDIA B200 (sm_100a).
 *
 * Pipeline of one layer (Alg. 1, forward pass; Fig. 1):
 *
 *   real activations --qnn_encode_pack--> activation bit planes  \
 *                                                                  qnn_bgemm / qnn_bconv2d --> fp32 outputs
 *   real weights ------qnn_pack_weights-> weight bit planes      /   (all plane pairs, 2^(i+j) combine, scale)
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.  The caller
 *     owns every buffer; the library allocates nothing, never frees, and never
 *     modifies an input.  The only state it keeps between calls is on the device:
 *     one status word that the tensor-path kernels set when a bounded wait gives
 *     up (read and cleared by qnn_tensor_path_status), and the fixed scratch array
 *     of qnn_fc_forward_noalloc; on the host, the per-device address of that array.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     only enqueue work; they return before it has run.
 *   - Every call returns a qnn_status.  Argument errors are found on the host
 *     before anything is enqueued; no exception or abort crosses this boundary.
 *   - Bit widths are 1..8.  "ab"/"wb" = activation / weight bits.
 *     A = 2^ab - 1 and B = 2^wb - 1 are the largest odd codes.
 *   - Mg, Ng, Kg = rows of activations, output features, reduction length.
 *
 * Encoding (Eq. 7, Section 3.2, Table 2).  A real x with grid step `scale`
 * (= r/(2^b - 1) for data in [-r, r]) becomes the odd integer q in
 * {-(2^b-1), ..., -1, +1, ..., 2^b-1} nearest to x/scale; a value half-way
 * between two codes goes to the one farther from zero, 0 goes to -1, values
 * outside [-r, r] take the end codes, NaN takes the most negative code.
 * q = sum_{i<b} 2^i c_i with c_i in {-1,+1}; with t = (q + 2^b - 1)/2, c_i = +1
 * exactly when bit i of t is 1.  Plane i stores c_i of every element, 1 bit each
 * (bit 1 means +1).
 *
 * Plane storage.  uint32 planes[row][plane i][word]; element k of a row is bit
 * (k mod 32) of word (k div 32); a row of k elements occupies
 * qnn_row_words(k) = ceil(k/32) rounded up to a multiple of 4 words per plane;
 * all padding bits are 0.  Plane buffers must be 16-byte aligned.
 */
#ifndef QNN_H
#define QNN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum qnn_status {
    QNN_OK = 0,
    QNN_E_ARG = -1,    /* null pointer, non-positive size, bits outside 1..8, unknown flag/layout */
    QNN_E_ALIGN = -2,  /* a plane/packed buffer is not 16-byte aligned, fp32 buffer not 4-byte aligned */
    QNN_E_RANGE = -3,  /* Kg*A*B does not fit int32, or an index does not fit the kernels' 32-bit tile arithmetic */
    QNN_E_SCALE = -4,  /* scale outside [1e-30, 1e30] (or NaN), or alpha not finite */
    QNN_E_CUDA = -5,   /* the CUDA runtime refused a launch or copy (cudaGetLastError is consumed) */
    QNN_E_DEVICE = -6  /* a kernel gave up a bounded wait (qnn_tensor_path_status) */
} qnn_status;

/* flags of qnn_encode_pack */
#define QNN_RELU 1u /* apply max(x, 0) before quantizing (the ReLU between layers of a stack) */

/* source layouts of qnn_pack_weights; element (n, tap, c) of the logical weight tensor is read from */
#define QNN_W_NTC 0 /* w[(n*taps + tap)*c_in + c]   : FC [Ng][Kg] (taps = 1) or conv [Cout][R][S][Cin] */
#define QNN_W_TCN 1 /* w[(tap*c_in + c)*n_out + n]  : FC stored k-major [Kg][Ng], conv [R][S][Cin][Cout] */
#define QNN_W_NCT 2 /* w[(n*c_in + c)*taps + tap]   : conv [Cout][Cin][R][S] */

const char *qnn_status_string(int status);
int qnn_version(void);

/* Words per (row, plane) for a row of k elements: ceil(k/32) rounded up to 4. */
size_t qnn_row_words(int64_t k);
/* Bytes of a plane buffer: rows * bits * qnn_row_words(k) * 4. */
size_t qnn_planes_bytes(int64_t rows, int64_t k, int bits);
/* Bytes of the packed-weights blob written by qnn_pack_weights (layout below). */
size_t qnn_weights_bytes(int n_out, int taps, int c_in, int bits);
/* Words per (output feature, plane) inside the packed-weights blob: taps*ceil(c_in/32) rounded up to 4. */
size_t qnn_weights_row_words(int taps, int c_in);

/*
 * Quantize, encode and bit-plane-pack activations in one pass (Eq. 7; Table 2;
 * the encoder stage of Fig. 1; Alg. 1 forward "MBitEncoder" step, evaluated
 * as the look-up form of Section 3.3).
 *   x       fp32 [rows][ldx], row r starts at x + r*ldx, first k entries used (ldx >= k).
 *           For a convolution input in NHWC, rows = N*H*W and k = C.
 *   scale   grid step s = r/(2^bits - 1), in [1e-30, 1e30] (QNN_E_SCALE otherwise).
 *   flags   0 or QNN_RELU.
 *   planes  out, uint32 [rows][bits][qnn_row_words(k)], fully written (padding = 0).
 *   rowsum  optional out (may be NULL), int32 [rows]: sum over the row of t = (q + 2^bits - 1)/2.
 */
int qnn_encode_pack(const float *x, int64_t rows, int k, int64_t ldx, int bits, float scale, unsigned flags,
                    uint32_t *planes, int32_t *rowsum, void *stream);

/*
 * Offline weight decomposition: quantize real weights to odd codes and store
 * their bit planes (Section 4.2: the quantized network's weights are
 * transformed into bit-encoded binary weights used at inference; Eq. 21).
 *   w        fp32, n_out*taps*c_in elements in one of the QNN_W_* layouts.
 *            FC: taps = 1, c_in = Kg.  Convolution: taps = R*S, c_in = Cin.
 *   packed   out, qnn_weights_bytes(...) bytes, 16-byte aligned:
 *              uint32 planes[n_out][bits][qnn_weights_row_words(taps, c_in)]
 *                 word tap*ceil(c_in/32) + c/32, bit c%32 holds element (tap, c);
 *                 each tap starts on a word boundary, padding bits are 0;
 *              followed by int32 tapsum[n_out][taps] = sum_c t(n, tap, c), which the
 *                 convolution needs for taps that fall outside the image.
 */
int qnn_pack_weights(const float *w, int n_out, int taps, int c_in, int layout, int bits, float scale,
                     void *packed, void *stream);

/*
 * Fully-connected layer on packed planes (Eq. 8 and Eq. 9; Alg. 1 forward,
 * the weighted branch sum and the scale): for every output (m, n)
 *   X_ij   = popcount over the row of (a_i[m] xor w_j[n])      for all ab*wb plane pairs,
 *   acc    = Kg*A*B - 2 * sum_ij 2^(i+j) X_ij                   (= sum_k q_a[m][k]*q_w[n][k], exact int32),
 *   out    = float(acc) * alpha                                 (alpha = scale_a * scale_w).
 * All pairs, the combine and the scale happen in one launch.
 *   a_planes  uint32 [Mg][ab][qnn_row_words(Kg)]
 *   w_packed  blob of qnn_pack_weights(n_out = Ng, taps = 1, c_in = Kg, bits = wb)
 *   out       fp32 [Mg][ldo] (ldo >= Ng), may be NULL if acc is given
 *   acc       optional int32 [Mg][Ng] (dense), the exact accumulators
 * QNN_E_RANGE if Kg*A*B >= 2^31.
 */
int qnn_bgemm(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg,
              float alpha, float *out, int64_t ldo, int32_t *acc, void *stream);

/*
 * Convolution lowered by implicit im2col onto the same plane-pair contraction
 * (Section 3.2: the decomposition applies to convolution layers as to
 * fully-connected ones; Eq. 9 applies the layer operation to the encoded
 * tensors).  The encoded activation tensor is padded with true zeros: a tap
 * outside the image adds nothing, so for each output pixel only the taps inside
 * the image are counted.
 *   a_planes  uint32 [N*H*W][ab][qnn_row_words(C)]   (NHWC pixels as rows)
 *   w_packed  blob of qnn_pack_weights(n_out = Cout, taps = R*S, c_in = C, bits = wb)
 *   out       fp32 [N][Ho][Wo][Cout], Ho = (H + 2*pad - R)/stride + 1, Wo likewise; may be NULL if acc given
 *   acc       optional int32, same shape as out
 */
int qnn_bconv2d(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C,
                int Cout, int R, int S, int stride, int pad, float alpha, float *out, int32_t *acc,
                void *stream);

/*
 * Dilated and transposed convolution on the same contraction (Section 3.2 names deconvolution layers next to
 * convolution layers).  Arguments as qnn_bconv2d, plus
 *   dilation    >= 1: tap (r, s) reads input (ho*stride - pad + r*dilation, wo*stride - pad + s*dilation)
 *   transposed  != 0: transposed convolution ("deconvolution"): every input pixel (hi, wi) contributes through tap
 *               (r, s) to output (hi*stride - pad + r*dilation, wi*stride - pad + s*dilation);
 *               Ho = (H-1)*stride - 2*pad + dilation*(R-1) + 1 + out_pad, Wo likewise; w_packed holds the weights
 *               as [Cout][R][S][Cin] of that scatter (no flipping is applied)
 *   out_pad     extra rows/columns of a transposed convolution's output (0 otherwise; < max(stride, dilation))
 * Forward: Ho = (H + 2*pad - dilation*(R-1) - 1)/stride + 1.  Positions outside the input (and, for the transposed
 * form, the zeros between its pixels) contribute nothing.  QNN_E_RANGE for geometries outside the tiled kernel.
 */
int qnn_bconv2d_general(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C,
                        int Cout, int R, int S, int stride, int pad, int dilation, int transposed, int out_pad,
                        float alpha, float *out, int32_t *acc, void *stream);

/*
 * Layer chaining (Alg. 1 forward: weighted branch sum, scale, then the next layer's MBitEncoder): the
 * contraction of qnn_bgemm / qnn_bconv2d whose epilogue can also apply a per-feature affine and quantize,
 * encode and bit-plane-pack its own fp32 result for the next layer, so that a stack of layers never
 * round-trips through fp32 in memory.
 *   ch_gamma, ch_beta   optional fp32 [Ng] (device): y = fma(float(acc)*alpha, ch_gamma[n], ch_beta[n]), one
 *                       rounding; a folded batch normalisation (Section 3.2: when batch normalisation follows,
 *                       the fixed scaling factor is not used, i.e. pass alpha = 1).  ch_beta may be NULL (0);
 *                       ch_gamma NULL = no affine.
 *   next_planes  optional out, uint32 [Mg][next_bits][qnn_row_words(Ng)] (conv: Mg = N*Ho*Wo pixels,
 *                Ng = Cout), bit-identical to qnn_encode_pack applied to the fp32 result y; NULL = no encoder
 *                (then next_bits / next_scale / next_flags are ignored)
 *   next_bits, next_scale, next_flags   as bits / scale / flags of qnn_encode_pack (QNN_RELU = the ReLU
 *                                       between the layers); the scale is fixed by the caller beforehand
 *                                       (the paper's range r is a constant or a learned parameter)
 *   out          optional fp32 result y; may be NULL when next_planes is given, except for convolutions whose
 *                whole patch fits one word (R*S*C <= 32) or whose geometry is outside the tiled kernel:
 *                those encode from `out` in a second launch and need it (the latter also take no affine)
 * At least one of ch_gamma / next_planes must be given.  Other arguments, checks and errors as in
 * qnn_bgemm / qnn_bconv2d.
 */
int qnn_bgemm_encode(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg,
                     float alpha, const float *ch_gamma, const float *ch_beta, int next_bits, float next_scale,
                     unsigned next_flags, uint32_t *next_planes, float *out, int64_t ldo, void *stream);
int qnn_bconv2d_encode(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int N, int H, int W, int C,
                       int Cout, int R, int S, int stride, int pad, float alpha, const float *ch_gamma,
                       const float *ch_beta, int next_bits, float next_scale, unsigned next_flags,
                       uint32_t *next_planes, float *out, void *stream);

/*
 * Training-side form of the encoder: the trigonometric M-bit encoder (Eq. 10) and its derivative (Eq. 12).
 * With xn = x / r and k_m = (2^bits - 1) / 2^m (m = 1..bits):
 *   forward   c[(m-1)*n + e] = phi^m(xn[e]) = sign(sin(k_m*pi*xn)) for m = bits, sign(-sin(k_m*pi*xn)) otherwise,
 *             as -1, 0 or +1 (0 exactly at a zero crossing).  The sign is taken from y = k_m*xn (one binary32
 *             product): 0 if y is an integer, else by the parity of floor(y); no library sine decides it.
 *             Away from the crossings these are the planes of qnn_encode_pack for data in [-r, r].
 *   backward  gx[e] = (1/r) * sum_m gc[(m-1)*n + e] * (+-) k_m*pi*cos(k_m*pi*xn[e]) for |xn| <= 1, else 0
 *             (+ for m = bits, - otherwise): the straight-through estimate of Eq. 12, in binary32.
 *   x fp32 [n]; c, gc fp32 [bits][n]; gx fp32 [n]; r in [1e-30, 1e30].
 */
int qnn_mbit_encoder_forward(const float *x, size_t n, int bits, float r, float *c, void *stream);
int qnn_mbit_encoder_backward(const float *x, const float *gc, size_t n, int bits, float r, float *gx, void *stream);

/*
 * Backward products of a fully-connected layer (Algorithm 1, backward propagation).  The forward is
 * a[r][n] = alpha * sum_k qa[r][k] * qw[n][k] with qa, qw the odd codes whose planes a^m, W^j the layer holds
 * (qa = sum_m 2^(m-1) a^m, qw = sum_j 2^(j-1) W^j).  Given g = dC/da, fp32 [m][n]:
 *   qnn_bgemm_backward_data     G [r][kk] = alpha * sum_nn g[r][nn] * qw[nn][kk];  Algorithm 1's per-plane gradient is
 *                               g_{a^p} = 2^(p-1) * G.  With x given (fp32 [m][k], the values the previous layer fed
 *                               to its encoder, range r, ab planes) the encoder derivative of Eq. 12 is applied in
 *                               the same kernel: out[r][kk] = (1/r) * sum_p 2^(p-1) * G[r][kk] * dphi^p/dxn(x[r][kk]/r),
 *                               i.e. qnn_mbit_encoder_backward fed with gc_p = 2^(p-1) * G.  x = NULL: out = G
 *                               (ab and r are ignored).
 *   qnn_bgemm_backward_weights  GW[nn][kk] = alpha * sum_r g[r][nn] * qa[r][kk];  g_{W^j} = 2^(j-1) * GW.
 * Both are TF32 tensor-core contractions with fp32 accumulation: the codes are exact, each element of g enters with
 * 11 significant bits, so |error| <= alpha * sum |g| * |q| * (2^-10 + contraction length * 2^-24); a g whose
 * elements have at most 11 significant bits and whose sums stay below 2^24 in units of its last place is contracted
 * exactly.
 *   w_planes  device planes [n][wb][qnn_row_words(k)] (what qnn_encode_pack writes for a [n][k] matrix; the
 *             canonical-plane view of packed FC weights), a_planes [m][ab][qnn_row_words(k)]; 16-byte aligned
 *   g         device fp32 [m][n], 16-byte aligned for backward_data (4-byte for backward_weights)
 *   out / gw  device fp32 [m][k] / [n][k]
 *   workspace device scratch owned by the caller, 256-byte aligned, at least qnn_bgemm_backward_*_workspace(m, n, k)
 *             bytes (0 from the query = dimensions out of range); holds the codes (and g) in the operand order the
 *             tensor cores read.  Every dimension is at most 65535*32.
 * QNN_E_ARG also for a workspace that is too small.  The kernels bound every wait on an arrival; one that gives up
 * is reported by qnn_tensor_path_status.
 */
size_t qnn_bgemm_backward_data_workspace(size_t m, size_t n, size_t k);
int qnn_bgemm_backward_data(const float *g, const uint32_t *w_planes, size_t m, size_t n, size_t k, int wb, float alpha,
                            const float *x, int ab, float r, float *out, void *workspace, size_t workspace_bytes,
                            void *stream);
size_t qnn_bgemm_backward_weights_workspace(size_t m, size_t n, size_t k);
int qnn_bgemm_backward_weights(const float *g, const uint32_t *a_planes, size_t m, size_t n, size_t k, int ab,
                               float alpha, float *gw, void *workspace, size_t workspace_bytes, void *stream);

/*
 * Backward products of a convolution layer (Algorithm 1, backward propagation, with forward() the convolution of
 * qnn_bconv2d: out[n][ho][wo][co] = alpha * sum_{r,s,c} qa[n][ho*stride - pad + r][wo*stride - pad + s][c] * qw[co][r][s][c],
 * taps outside the image contributing nothing).  Given g = dC/d(out), fp32 [N][Ho][Wo][Cout]:
 *   qnn_bconv2d_backward_data     G[n][h][w][c] = alpha * sum over (co, r, s) and the output pixels that read input
 *                                 pixel (h, w) through tap (r, s) of g[n][ho][wo][co] * qw[co][r][s][c]; Algorithm 1's
 *                                 per-plane gradient is g_{a^p} = 2^(p-1) * G.  x (optional, fp32 [N][H][W][C], with ab
 *                                 and r) applies the encoder derivative of Eq. 12 as in qnn_bgemm_backward_data.
 *   qnn_bconv2d_backward_weights  GW[co][r][s][c] = alpha * sum over the output pixels of g[n][ho][wo][co] *
 *                                 qa[n][ho*stride - pad + r][wo*stride - pad + s][c]; g_{W^j} = 2^(j-1) * GW.
 * Both are TF32 tensor-core contractions like the fully-connected products.  The data gradient is an implicit GEMM over
 * (tap, output feature): the kernel gathers its operand from g itself, one shifted box per tap, so no patch matrix is
 * ever written and each result element is a single fp32 accumulation of R*S*Cout terms; the workspace only holds the
 * unpacked weight codes (and a row-padded copy of g when Cout is not a multiple of 4).  The weight gradient contracts
 * over the output pixels; it too is an implicit GEMM, on the transposed gradient and S*stride copies of the transposed
 * activation codes with the stride and the shift along w baked in (tap rows are shifts of the box that the kernel
 * reads), which the call stages in the workspace (at stride 1 about 1 + S times the layer's tensors in fp32); where those
 * copies would not be clearly smaller than the im2col of the codes ([R*S*C][N*Ho*Wo] fp32; e.g. 3 x 3 at stride 2) it
 * stages that instead.  Error bound as for the fully-connected products with contraction lengths
 * R*S*Cout (data) and N*Ho*Wo (weights, plus the columns that pad each image row to a multiple of 4, which add exact
 * zeros); integer-valued g with small sums is contracted exactly.
 *   w_packed  blob of qnn_pack_weights(n_out = Cout, taps = R*S, c_in = C, bits = wb); a_planes [N*H*W][ab][qnn_row_words(C)]
 *   g         device fp32, 16-byte aligned for backward_data (4-byte for backward_weights)
 *   out / gw  device fp32 [N][H][W][C] / [Cout][R][S][C]
 *   workspace device scratch owned by the caller, 256-byte aligned, at least qnn_bconv2d_backward_*_workspace(...)
 *             bytes (0 from the query = geometry out of range: N*Ho*Wo, R*S*C and Cout at most 65535*32,
 *             R*S*ceil(C/32) at most 65535).
 * The weight gradients (convolution and fully-connected) split a long contraction over the thread blocks when the result
 * has few tiles and add the partial products in a fixed order: results repeat bit for bit from call to call.
 * Errors as for qnn_bgemm_backward_*; waits are bounded and reported by qnn_tensor_path_status.
 */
size_t qnn_bconv2d_backward_data_workspace(int N, int H, int W, int C, int Cout, int R, int S, int stride, int pad);
int qnn_bconv2d_backward_data(const float *g, const void *w_packed, int wb, int N, int H, int W, int C, int Cout, int R,
                              int S, int stride, int pad, float alpha, const float *x, int ab, float r, float *out,
                              void *workspace, size_t workspace_bytes, void *stream);
size_t qnn_bconv2d_backward_weights_workspace(int N, int H, int W, int C, int Cout, int R, int S, int stride, int pad);
int qnn_bconv2d_backward_weights(const float *g, const uint32_t *a_planes, int ab, int N, int H, int W, int C, int Cout,
                                 int R, int S, int stride, int pad, float alpha, float *gw, void *workspace,
                                 size_t workspace_bytes, void *stream);

/*
 * Planes [rows][bits][qnn_row_words(k)] -> the odd codes q = sum_i 2^(i-1) * plane_i (Eq. 8) as fp32:
 * out[row*ld + col] (transpose = 0, ld >= k) or out[col*ld + row] (transpose != 0, ld >= rows).
 */
int qnn_unpack_codes_f32(const uint32_t *planes, size_t rows, size_t k, int bits, int transpose, float *out, size_t ld,
                         void *stream);

/*
 * Synchronises the device and reports whether a tensor-path kernel gave up a bounded wait since the last call:
 * *status = 0 and QNN_OK, or *status = 1 + the id of the first wait that gave up (0 producer waiting for a free
 * stage, 1 MMA issuer waiting for a stage's operands, 2 epilogue waiting for an accumulator, 3 MMA issuer waiting
 * for a free accumulator buffer) and QNN_E_DEVICE; the record is cleared.  Results of a call that reported an
 * error are undefined (its kernels have ended and released what they held; the context stays usable).
 * qnn_last_device_status is the same call under the name the status word has in the library's error convention.
 */
int qnn_tensor_path_status(unsigned int *status);
int qnn_last_device_status(unsigned int *status);

/*
 * Self-test of the bounded waits (no counterpart in the paper; diagnostic only).  Enqueues one small thread block
 * built from the tensor-path kernels' own wait helpers in which a producer waits for a stage release that never
 * comes: after poll_limit polls (16..65536) it gives up, raises the block's abort flag and the library's status
 * word with wait id 0, lets its copy in flight land, and a second warp waiting for an accumulator leaves through the
 * abort flag.  The kernel then ends normally -- nothing traps, faults or spins without bound.  The next
 * qnn_tensor_path_status call therefore returns QNN_E_DEVICE with *status = 1 and clears the record; later calls
 * of the library are unaffected.
 */
int qnn_selftest_bounded_wait(unsigned int poll_limit, void *stream);

/*
 * Comparison only, not the paper's method: the product of qnn_bgemm computed as ONE signed 8-bit tensor-core GEMM
 * on the unpacked odd codes (Eq. 8 read backwards: q = sum_i 2^(i-1) * plane_i), to show what the bit-plane
 * decomposition competes with on this GPU.  Arguments as qnn_bgemm (a_planes, w_packed of a fully-connected layer
 * with taps = 1, alpha); acc (optional) receives the int32 accumulators [Mg][Ng], out (optional) float(acc) * alpha;
 * at least one of them is given.  Both are bit-identical to qnn_bgemm's.  ab, wb <= 7 (QNN_E_RANGE for 8: the code
 * +-255 does not fit a signed byte), Kg*A*B < 2^31.  workspace: device scratch of at least
 * qnn_bgemm_int8_tensor_workspace(Mg, Ng, Kg) bytes, 256-byte aligned, owned by the caller (holds the unpacked codes).
 */
size_t qnn_bgemm_int8_tensor_workspace(int64_t Mg, int Ng, int Kg);
int qnn_bgemm_int8_tensor(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng, int Kg,
                          float alpha, int32_t *acc, float *out, void *workspace, size_t workspace_bytes, void *stream);

/*
 * max_i |x[i]| into *out (device fp32), for workloads whose grid step is derived
 * from the tensor's range.  Not a step of the paper's method (its range r is a
 * fixed or learned constant, Eq. 9 / Eq. 15).  NaNs are ignored.
 */
int qnn_absmax_f32(const float *x, size_t n, float *out, void *stream);

/*
 * One FC layer from host memory: copies x_host to x_dev, runs qnn_encode_pack
 * and qnn_bgemm, copies the fp32 result to out_host, all on `stream`.
 * Device work buffers are the caller's: x_dev [Mg*Kg] fp32, planes_dev
 * qnn_planes_bytes(Mg, Kg, ab), out_dev [Mg*Ng] fp32.  x_host / out_host should be
 * pinned for the copies to be asynchronous.  The result is in out_host once the
 * stream has been synchronized.
 */
int qnn_fc_forward_host(const float *x_host, int64_t Mg, int Kg, int ab, float scale_a, unsigned flags,
                        const void *w_packed, int wb, int Ng, float alpha, float *out_host, float *x_dev,
                        uint32_t *planes_dev, float *out_dev, void *stream);

/*
 * The same layer from host memory, cut into chunks of `rows_per_chunk` activation rows that are spread
 * round-robin over `nstreams` caller-provided streams (cudaStream_t each): chunk i is copied in, encoded,
 * contracted and copied out on stream i % nstreams, so the two copy directions and the kernels of different
 * chunks overlap (rows are independent).  Buffers as in qnn_fc_forward_host (each chunk uses its own row
 * range of them).  The caller orders the streams against earlier and later work; out_host is complete once
 * every stream has been synchronized.
 */
int qnn_fc_forward_host_pipelined(const float *x_host, int64_t Mg, int Kg, int ab, float scale_a, unsigned flags,
                                  const void *w_packed, int wb, int Ng, float alpha, float *out_host, float *x_dev,
                                  uint32_t *planes_dev, float *out_dev, int64_t rows_per_chunk, void *const *streams,
                                  int nstreams);

/*
 * One FC layer for callers that cannot allocate device memory.  (The paper has no counterpart: this is a
 * packaging of qnn_encode_pack + qnn_bgemm, not a step of the method.)
 *
 * Some callers only ever hold the pointers they were given: a plug-in callback inside a host framework
 * that owns all device memory and forbids allocation from callbacks, a real-time loop whose memory was
 * fixed at start-up, a plain C program without an allocator.  They cannot supply the activation-planes
 * buffer that sits between the encoder and the contraction.  This call keeps that buffer inside the
 * library, as a fixed array of QNN_NOALLOC_SCRATCH_BYTES in the GPU's global memory (each GPU that loads
 * the library holds it until the process exits), and calls neither cudaMalloc nor cudaFree nor any
 * routine that allocates.
 *
 *   x         fp32 [Mg][ldx] (device), first Kg entries of each row used
 *   w_packed  blob of qnn_pack_weights(n_out = Ng, taps = 1, c_in = Kg, bits = wb) (device)
 *   out       fp32 [Mg][ldo] (device), ldo >= Ng
 * Computes exactly what qnn_encode_pack followed by qnn_bgemm computes (same kernels, same bits).
 *
 * Limit: qnn_planes_bytes(Mg, Kg, ab) must not exceed QNN_NOALLOC_SCRATCH_BYTES (e.g. 4096 x 4096 at
 * up to 4 bits, or 16384 x 4096 at 1 bit); larger problems are refused with QNN_E_RANGE before anything
 * is enqueued.  Other argument errors are reported as by the two underlying calls.
 *
 * First call on a device: the library looks up the device address of its array once per device, with
 * that device current (a host-side runtime query, no allocation).  Make that first call outside any
 * stream capture; later calls only enqueue the two kernels on `stream`.
 *
 * Sharing: every call on a device uses the same array and leaves its planes there.  Nothing needs to
 * start at zero (the encoder overwrites every word it will read, padding included), so consecutive calls
 * on one stream are safe; two calls whose kernels can overlap on the GPU (different streams, or different
 * host threads on different streams) race on the array and must be ordered by the caller.
 */
#define QNN_NOALLOC_SCRATCH_BYTES (8u << 20)
int qnn_fc_forward_noalloc(const float *x, int64_t Mg, int Kg, int64_t ldx, int ab, float scale_a, unsigned flags,
                           const void *w_packed, int wb, int Ng, float alpha, float *out, int64_t ldo, void *stream);

/*
 * Peak probes used to state a roofline next to a measurement.
 * qnn_probe_bitops enqueues a register-resident kernel that does nothing but the
 * contraction's instruction mix and returns (in *word_ops) how many 32-bit
 * xor-popcount-accumulate word operations it performs; divide by its measured time.
 *   variant 0: xor + popc + add per word, operands in registers (this is popcount-issue bound and so
 *              measures the popcount pipe: one popcount per word);
 *   variant 1: the 3:2 carry-save form in registers (3 xor, 2 three-input logic ops, 2 popc per 3 words);
 *   variant 2: the tiled kernel's own inner loop (7:3 bit-column counters on re-coded operands: 8 xor,
 *              5 three-input logic ops, 4 popc, 4 multiply-adds per 8 words) fed from shared memory;
 *   variant 3 / 4: warp-level 1-bit tensor-core instruction mma.sync m16n8k256 with and.popc / xor.popc,
 *              operands in registers (word_ops counts 32 binary multiply-accumulates as one word operation).
 *   sink: device int32 [blocks*256], written once at the end.
 * qnn_probe_copy enqueues a plain 16-byte-vector device copy of `bytes` (multiple of 16).
 * qnn_popcounts_per_output returns how many popcount instructions the kernel that qnn_bgemm (is_conv = 0, R = S = 1,
 * C = Kg, Cout = Ng) or qnn_bconv2d (is_conv != 0) runs for such a layer issues per output element, all ab*wb plane
 * pairs together (0 = arguments out of range): the popcount pipe is the scarce unit of the contraction, so
 * outputs * that number / the popcount rate of probe variant 0 is the layer's bit-operation roofline time.
 * qnn_probe_naive_sgemm enqueues the plain fp32 product that the efficiency experiment (Section 5.4, Fig. 7, Eq. 16)
 * sets the bit-plane product against: c[m][n] = sum_k a[m][k] * b[k][n], device pointers, all three row-major and
 * dense, one thread per output, one fused multiply-add per reduction step in increasing k, nothing tiled.  A
 * comparison line only: no product path calls it.  QNN_E_ARG on null pointers or sizes <= 0, QNN_E_RANGE when
 * m > 8 * 65535.
 */
int qnn_probe_bitops(int variant, int iters, int blocks, int32_t *sink, double *word_ops, void *stream);
int qnn_probe_naive_sgemm(const float *a, const float *b, float *c, int m, int n, int k, void *stream);
int64_t qnn_popcounts_per_output(int ab, int wb, int is_conv, int R, int S, int C, int Cout);
int qnn_probe_copy(void *dst, const void *src, size_t bytes, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* QNN_H */

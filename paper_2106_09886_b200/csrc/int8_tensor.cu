// Comparison path, not the method: the forward product of a layer computed as ONE int8 tensor-core GEMM on the
// unpacked odd codes (q = sum_i 2^i * plane_i, Eq. 8), i.e. what the {-1,+1} bit-plane decomposition competes with on
// this GPU.  Same integer result as qnn_bgemm (int32 accumulators, then float(acc) * alpha), same persistent tcgen05
// skeleton as the backward products with kind::i8 and an int32 accumulator in tensor memory.  Codes of up to 7 bits fit
// a signed byte.
#include "tc_gemm.cuh"

namespace {

// Bit planes [rows][BITS][kw] -> int8 codes out[row][ld].  A warp writes 128 codes (128 bytes) of one row per step:
// lane -> plane word lane/8 of a group of four, bits [4*(lane%8), +4) of it, stored as one char4.
template <int BITS>
__global__ void __launch_bounds__(256) unpack_codes_i8_kernel(const uint32_t *__restrict__ planes, long long rows, long long k,
                                                             long long kw, int8_t *__restrict__ out, long long ld) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long word = (long long)blockIdx.x * 4 + (lane >> 3);
    const int sh = 4 * (lane & 7);
    const long long col = word * 32 + sh;
    constexpr int amax = (1 << BITS) - 1;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long row = (long long)blockIdx.y * 32 + warp + 8 * i;
        if (row >= rows || col >= k) continue;
        int t[4] = {0, 0, 0, 0};
#pragma unroll
        for (int b = 0; b < BITS; ++b) {
            const uint32_t w = __ldg(planes + (row * BITS + b) * kw + word) >> sh;
#pragma unroll
            for (int e = 0; e < 4; ++e) t[e] |= (int)((w >> e) & 1u) << b;
        }
        char4 q;
        q.x = (signed char)(2 * t[0] - amax);
        q.y = (signed char)(2 * t[1] - amax);
        q.z = (signed char)(2 * t[2] - amax);
        q.w = (signed char)(2 * t[3] - amax);
        // columns at and beyond k are never read (the tensor map ends at k), so a partly valid group may be written whole
        *reinterpret_cast<char4 *>(out + row * ld + col) = q;
    }
}

int unpack_i8(const uint32_t *planes, long long rows, long long k, int bits, int8_t *out, long long ld, cudaStream_t st) {
    const long long kw = qnn_row_words_i(k);
    const dim3 grid((unsigned)(kw / 4), (unsigned)qnn_ceil_div(rows, 32));
#define UNPACK_CASE(B) case B: unpack_codes_i8_kernel<B><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    switch (bits) {
        UNPACK_CASE(1) UNPACK_CASE(2) UNPACK_CASE(3) UNPACK_CASE(4) UNPACK_CASE(5) UNPACK_CASE(6)
        default: unpack_codes_i8_kernel<7><<<grid, 256, 0, st>>>(planes, rows, k, kw, out, ld); break;
    }
#undef UNPACK_CASE
    return qnn_launch_status();
}

long long pad128(long long v) { return (v + 127) / 128 * 128; }

bool i8_dims_ok(int64_t Mg, int Ng, int Kg) {
    const int64_t lim = (int64_t)65535 * 32;
    return Mg >= 1 && Ng >= 1 && Kg >= 1 && Mg <= lim && Ng <= lim && Kg <= lim;
}

}  // namespace

extern "C" size_t qnn_bgemm_int8_tensor_workspace(int64_t Mg, int Ng, int Kg) {
    if (!i8_dims_ok(Mg, Ng, Kg)) return 0;
    return (size_t)(Mg + Ng) * (size_t)pad128(Kg);
}

extern "C" int qnn_bgemm_int8_tensor(const uint32_t *a_planes, int ab, const void *w_packed, int wb, int64_t Mg, int Ng,
                                     int Kg, float alpha, int32_t *acc, float *out, void *workspace,
                                     size_t workspace_bytes, void *stream) {
    if (!a_planes || !w_packed || !workspace || (!acc && !out) || !i8_dims_ok(Mg, Ng, Kg) || !qnn_bits_ok(ab) ||
        !qnn_bits_ok(wb))
        return QNN_E_ARG;
    if (ab > 7 || wb > 7) return QNN_E_RANGE;                         // an 8-bit odd code reaches +-255
    if ((double)Kg * ((1 << ab) - 1) * ((1 << wb) - 1) >= 2147483648.0) return QNN_E_RANGE;
    if (!(fabsf(alpha) <= 3.0e38f)) return QNN_E_SCALE;
    if (workspace_bytes < qnn_bgemm_int8_tensor_workspace(Mg, Ng, Kg)) return QNN_E_ARG;
    if (!qnn_aligned(a_planes, 16) || !qnn_aligned(w_packed, 16) || !qnn_aligned(workspace, 256) ||
        (acc && !qnn_aligned(acc, 4)) || (out && !qnn_aligned(out, 4)))
        return QNN_E_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long ld = pad128(Kg);
    int8_t *qa = static_cast<int8_t *>(workspace);                     // [Mg][ld]
    int8_t *qw = qa + (size_t)Mg * ld;                                 // [Ng][ld]
    int rc = unpack_i8(a_planes, Mg, Kg, ab, qa, ld, st);
    if (rc != QNN_OK) return rc;
    // the packed weights of a fully-connected layer begin with the planes [Ng][wb][row words]
    if ((rc = unpack_i8(static_cast<const uint32_t *>(w_packed), Ng, Kg, wb, qw, ld, st)) != QNN_OK) return rc;
    GemmParams p{};
    p.M = (int)Mg; p.N = Ng; p.K = Kg;
    p.alpha = alpha;
    p.C = out; p.acc = acc; p.ldc = Ng;
    if (!(p.err = qnn_tc_error_word())) return QNN_E_CUDA;
    return run_gemm<TC_I8>(qa, ld, qw, ld, p, st);
}

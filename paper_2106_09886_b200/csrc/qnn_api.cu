// Status strings, version and size queries of libqnn.
#include "qnn_internal.cuh"

extern "C" const char *qnn_status_string(int status) {
    switch (status) {
        case QNN_OK: return "ok";
        case QNN_E_ARG: return "invalid argument (null pointer, size, bit width, flag or layout)";
        case QNN_E_ALIGN: return "buffer not aligned (planes and packed weights need 16 bytes)";
        case QNN_E_RANGE: return "size out of range (int32 accumulator or index arithmetic would overflow)";
        case QNN_E_SCALE: return "scale not finite or not positive";
        case QNN_E_CUDA: return "CUDA runtime error on launch or copy";
        case QNN_E_DEVICE: return "kernel reported an internal error";
        default: return "unknown status";
    }
}

extern "C" int qnn_version(void) { return QNN_VERSION_NUMBER; }

extern "C" size_t qnn_row_words(int64_t k) { return k <= 0 ? 0 : (size_t)qnn_row_words_i(k); }

extern "C" size_t qnn_planes_bytes(int64_t rows, int64_t k, int bits) {
    if (rows <= 0 || k <= 0 || !qnn_bits_ok(bits)) return 0;
    return (size_t)rows * (size_t)bits * (size_t)qnn_row_words_i(k) * 4u;
}

extern "C" size_t qnn_weights_row_words(int taps, int c_in) {
    if (taps <= 0 || c_in <= 0) return 0;
    return (size_t)qnn_w_row_words_i(taps, c_in);
}

extern "C" size_t qnn_weights_bytes(int n_out, int taps, int c_in, int bits) {
    if (n_out <= 0 || taps <= 0 || c_in <= 0 || !qnn_bits_ok(bits)) return 0;
    size_t planes = (size_t)n_out * (size_t)bits * (size_t)qnn_w_row_words_i(taps, c_in) * 4u;
    size_t tapsum = (size_t)n_out * (size_t)taps * 4u;
    return planes + (tapsum + 15u) / 16u * 16u;
}

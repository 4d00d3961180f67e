// Short-reduction kernels (Kg <= 128) for 2-bit activations, every weight width 1..4 and 1..4 words per plane.
#include "bconv_pointwise.cuh"

namespace qnn_pointwise {
int run_pointwise_ab2(int wb, int kw, const Params &p, cudaStream_t st) { return run_ab<2>(wb, kw, p, st); }
}  // namespace qnn_pointwise

// Instantiations of the tiled contraction for 7-bit activations, convolution operand (all weight widths).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab7_conv(int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<7, 1>(wb, p, st); }
}  // namespace qnn_tiled

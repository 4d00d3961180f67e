// Instantiations of the tiled contraction for 6-bit activations, dilated / transposed convolution operand (all weight widths).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab6_gconv(int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<6, 2>(wb, p, st); }
}  // namespace qnn_tiled

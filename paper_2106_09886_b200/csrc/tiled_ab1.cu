// Instantiations of the tiled contraction for 1-bit activations (all weight widths, FC and convolution).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab1(bool conv, int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<1>(conv, wb, p, st); }
}  // namespace qnn_tiled

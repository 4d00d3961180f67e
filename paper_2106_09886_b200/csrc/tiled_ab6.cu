// Instantiations of the tiled contraction for 6-bit activations (all weight widths, FC and convolution).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab6(bool conv, int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<6>(conv, wb, p, st); }
}  // namespace qnn_tiled

// Instantiations of the tiled contraction for 5-bit activations, fully-connected operand (all weight widths).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab5_fc(int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<5, 0>(wb, p, st); }
}  // namespace qnn_tiled

// Instantiations of the tiled contraction for 4-bit activations, fully-connected operand (all weight widths).
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_ab4_fc(int wb, const Params &p, cudaStream_t st) { return run_tiled_ab<4, 0>(wb, p, st); }
}  // namespace qnn_tiled

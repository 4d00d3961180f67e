// Instantiations of the tiled contraction for 3x3 convolutions with 9-word groups, 1-bit activations, weight widths 1..4.
#include "bgemm_tiled.cuh"

namespace qnn_tiled {
int run_tiled_conv3x3_ab1(int wb, const Params &p, cudaStream_t st) {
    switch (wb) {
        case 1: return launch_tiled<1, 1, 3>(p, st);
        case 2: return launch_tiled<1, 2, 3>(p, st);
        case 3: return launch_tiled<1, 3, 3>(p, st);
        case 4: return launch_tiled<1, 4, 3>(p, st);
        default: return QNN_E_ARG;
    }
}
}  // namespace qnn_tiled

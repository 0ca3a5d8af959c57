// Instances of the warp-level tensor-core convolution kernel: 16 channels per shared-memory row, 3xTF32.
#include "conv_mma.cuh"

namespace small {
namespace mma_conv {

MmaKernel pick_mma_16_x3(int NF, int FW, int S, bool vert) { return pick_mma_nf<16, true>(NF, FW, S, vert); }

}  // namespace mma_conv
}  // namespace small

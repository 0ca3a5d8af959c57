// Instances of the warp-level tensor-core convolution kernel: 32 channels per shared-memory row, 3xTF32.
#include "conv_mma.cuh"

namespace small {
namespace mma_conv {

MmaKernel pick_mma_32_x3(int NF, int FW, int S, bool vert) { return pick_mma_nf<32, true>(NF, FW, S, vert); }

}  // namespace mma_conv
}  // namespace small

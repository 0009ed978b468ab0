// Bit-serial convolution kernels for 3-bit activations (all weight widths and pixel-block sizes).
#include "conv_launch.cuh"

namespace bs {
int launch_conv_a3(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    return launch_conv_a<3>(WB, PB, args, grid, block, smem, st);
}
}  // namespace bs

// Bit-serial convolution kernels for 2-bit activations (all weight widths and pixel-block sizes).
#include "conv_launch.cuh"

namespace bs {
int launch_conv_a2(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    return launch_conv_a<2>(WB, PB, args, grid, block, smem, st);
}
}  // namespace bs

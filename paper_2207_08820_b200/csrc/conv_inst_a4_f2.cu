// Bit-serial convolution kernels: 4-bit activations, 2 filters per thread (all weight widths and pixel blocks).
#include "conv_launch.cuh"

namespace bs {
int launch_conv_a4_f2(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    return launch_conv_a<4, 2>(WB, PB, args, grid, block, smem, st);
}
}  // namespace bs

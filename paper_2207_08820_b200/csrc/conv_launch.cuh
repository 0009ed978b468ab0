// Instantiation helper: one translation unit per activation bit-width keeps compile times parallel.
#pragma once
#include "conv_kernel.cuh"

namespace bs {

constexpr int CONV_FB = 8;

template <int A, int WB, int PB>
inline int launch_conv_one(const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    auto kern = bitserial_conv_kernel<A, WB, PB, CONV_FB>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
            cudaGetLastError();
            return BS_ERR_CUDA;
        }
    }
    kern<<<grid, block, smem, st>>>(args);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

template <int A, int WB>
inline int launch_conv_pb(int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    switch (PB) {
        case 8: return launch_conv_one<A, WB, 8>(args, grid, block, smem, st);
        case 7: return launch_conv_one<A, WB, 7>(args, grid, block, smem, st);
        case 4: return launch_conv_one<A, WB, 4>(args, grid, block, smem, st);
        default: return BS_ERR_UNSUPPORTED;
    }
}

template <int A>
inline int launch_conv_a(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    switch (WB) {
        case 1: return launch_conv_pb<A, 1>(PB, args, grid, block, smem, st);
        case 2: return launch_conv_pb<A, 2>(PB, args, grid, block, smem, st);
        case 3: return launch_conv_pb<A, 3>(PB, args, grid, block, smem, st);
        case 4: return launch_conv_pb<A, 4>(PB, args, grid, block, smem, st);
        default: return BS_ERR_UNSUPPORTED;
    }
}

// defined in conv_inst_a{1,2,3,4}.cu
int launch_conv_a1(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st);
int launch_conv_a2(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st);
int launch_conv_a3(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st);
int launch_conv_a4(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st);

}  // namespace bs

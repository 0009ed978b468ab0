// Instantiation helper: one translation unit per activation bit-width keeps compile times parallel.
#pragma once
#include "conv_kernel.cuh"

namespace bs {

template <int A, int WB, int PB, int FB>
inline int launch_conv_one(const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    auto kern = bitserial_conv_kernel<A, WB, PB, FB>;
    if (smem > 48 * 1024) {
        if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)) != cudaSuccess) {
            cudaGetLastError();
            return BS_ERR_CUDA;
        }
    }
    kern<<<grid, block, smem, st>>>(args);
    return cudaGetLastError() == cudaSuccess ? BS_OK : BS_ERR_CUDA;
}

// (pixels per thread, filters per thread) pairs that are instantiated
#define BS_TILE_LIST(X) X(8, 8) X(7, 8) X(4, 8) X(8, 4) X(7, 4) X(4, 4) X(8, 2) X(7, 2) X(4, 2)

template <int A, int WB, int FB>
inline int launch_conv_pb(int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    // the filter block is a compile-time choice of the translation unit: only its own kernels are instantiated
#define BS_CASE(P_, F_) if constexpr (FB == F_) { if (PB == P_) return launch_conv_one<A, WB, P_, F_>(args, grid, block, smem, st); }
    BS_TILE_LIST(BS_CASE)
#undef BS_CASE
    return BS_ERR_UNSUPPORTED;
}

template <int A, int FB>
inline int launch_conv_a(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st)
{
    switch (WB) {
        case 1: return launch_conv_pb<A, 1, FB>(PB, args, grid, block, smem, st);
        case 2: return launch_conv_pb<A, 2, FB>(PB, args, grid, block, smem, st);
        case 3: return launch_conv_pb<A, 3, FB>(PB, args, grid, block, smem, st);
        case 4: return launch_conv_pb<A, 4, FB>(PB, args, grid, block, smem, st);
        default: return BS_ERR_UNSUPPORTED;
    }
}

// defined in conv_inst_a{1,2,3,4}_f{2,4,8}.cu
#define BS_DECLARE_CONV_LAUNCH(A, FB) \
    int launch_conv_a##A##_f##FB(int WB, int PB, const ConvArgs& args, unsigned grid, unsigned block, size_t smem, cudaStream_t st);
BS_DECLARE_CONV_LAUNCH(1, 2) BS_DECLARE_CONV_LAUNCH(1, 4) BS_DECLARE_CONV_LAUNCH(1, 8) BS_DECLARE_CONV_LAUNCH(2, 2) BS_DECLARE_CONV_LAUNCH(2, 4) BS_DECLARE_CONV_LAUNCH(2, 8)
BS_DECLARE_CONV_LAUNCH(3, 2) BS_DECLARE_CONV_LAUNCH(3, 4) BS_DECLARE_CONV_LAUNCH(3, 8) BS_DECLARE_CONV_LAUNCH(4, 2) BS_DECLARE_CONV_LAUNCH(4, 4) BS_DECLARE_CONV_LAUNCH(4, 8)
#undef BS_DECLARE_CONV_LAUNCH

}  // namespace bs

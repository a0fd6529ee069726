// Launchers of kernels that live in translation units of their own.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

// fp32, K <= 64: persistent tcgen05 kernel that streams D (skinny_umma_kernel.cuh)
constexpr int kSkinnyMaxK = 64;
cudaError_t launch_skinny_umma(const TiledParams &p, int ctas, cudaStream_t stream);

}  // namespace btc

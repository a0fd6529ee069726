// Launchers of kernels that live in translation units of their own.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

// fp32, K <= 64: persistent tcgen05 kernel that streams D (skinny_umma_kernel.cuh)
constexpr int kSkinnyMaxK = 64;
cudaError_t launch_skinny_umma(const TiledParams &p, const SkinnyBatch &batch, int ctas, cudaStream_t stream);

// any element type (0 fp32, 1 fp64, 2 complex64, 3 complex128), K <= 4: one thread per 16 bytes of D
// (stream_kernel.cuh).  vec_d: groups of 16 bytes along the first M mode are contiguous and aligned in D
// and C; vec_a: in A as well.
constexpr int kStreamVariant = 100;     // reported through BTC_ATTR_VARIANT / BTC_STATUS_VARIANT for every element type
constexpr int kStreamMaxContracted = 4;
cudaError_t launch_stream(const TiledParams &p, int dtype, bool vec_d, bool vec_a, int sm_count, cudaStream_t stream);

}  // namespace btc

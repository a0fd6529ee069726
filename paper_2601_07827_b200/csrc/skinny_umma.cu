// Translation unit of the short-K streaming kernel (fp32 on tcgen05).
#include "skinny_umma_kernel.cuh"

#include <atomic>

#include "launchers.h"

namespace btc {

cudaError_t launch_skinny_umma(const TiledParams &p, int ctas, cudaStream_t stream)
{
    static std::atomic<bool> configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_relaxed)) {
        cudaError_t e = cudaFuncSetAttribute(skinny_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(SkinnyTile::SMEM_BYTES));
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_relaxed);
    }
    skinny_umma_kernel<<<unsigned(ctas), SkinnyTile::THREADS, SkinnyTile::SMEM_BYTES, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace btc

// Translation unit of the short-K streaming kernel (fp32 on tcgen05).
#include "skinny_umma_kernel.cuh"

#include <atomic>

#include "launchers.h"

namespace btc {

cudaError_t launch_skinny_umma(const TiledParams &p, const SkinnyBatch &batch, int ctas, cudaStream_t stream)
{
    static std::atomic<bool> configured[64] = {};
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_relaxed)) {
        cudaError_t e = cudaFuncSetAttribute(skinny_umma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(SkinnyTile::SMEM_BYTES));
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_relaxed);
    }
    // Programmatic dependent launch: when the launch before this one in the stream is a kernel too, this
    // grid's CTAs may start (set-up only: tables of the operation, barriers, tensor memory) while that
    // kernel's last CTAs finish; the kernel waits for the earlier grid before it touches operand data.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(unsigned(ctas)); cfg.blockDim = dim3(SkinnyTile::THREADS);
    cfg.dynamicSmemBytes = SkinnyTile::SMEM_BYTES; cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, skinny_umma_kernel, p, batch);
}

}  // namespace btc

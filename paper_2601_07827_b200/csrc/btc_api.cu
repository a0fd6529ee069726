// C-ABI entry points of the contraction library (declared in include/btc.h): object management,
// tile/split-K choice and kernel launches.  No compute happens on the host.
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <climits>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/btc.h"
#include "generic_kernel.cuh"
#include "kernel_params.h"
#include "launchers.h"
#include "skinny_layout.h"
#include "plan.h"
#include "tiled_f32_kernel.cuh"
#include "tiled_f64_kernel.cuh"
#include "tiled_tf32x3_kernel.cuh"
#include "tiled_umma_tf32x3_kernel.cuh"
#include "isolated_sum_kernel.cuh"
#include "complex_expand_kernel.cuh"
#include "elementwise_kernels.cuh"

using namespace btc;


struct btc_handle_s {
    int device = -1;       // -1: no CUDA device (objects can be validated and planned, not run)
    int sm_count = 148;
};

struct btc_tensor_info_s {
    TensorDesc desc;
};

struct btc_status_s {
    int32_t kernel = 0, launches = 0, split_k = 1, variant = -1;
    int32_t grid[3] = {0, 0, 0};
};

struct btc_contraction_s {
    btc_handle_s handle;
    PlanRequest req;
    Plan plan;
    double alpha[2] = {1.0, 0.0}, beta[2] = {0.0, 0.0};
    // device copies of the plan's tables (one allocation)
    int64_t *d_tables = nullptr;
    int32_t *d_error = nullptr;   // inside d_tables' allocation; non-zero after a device-side wait gave up
    const int64_t *d_offA_m = nullptr, *d_offD_m = nullptr, *d_offB_n = nullptr, *d_offD_n = nullptr,
                  *d_offA_k = nullptr, *d_offB_k = nullptr, *d_offA_h = nullptr, *d_offB_h = nullptr,
                  *d_offD_h = nullptr;
    int32_t tiles_m = 0, tiles_n = 0, raster_n_fast = 0;
    int64_t k_per_split = 0;
    // bulk-tensor-copy variants: the M-side operand as a tensor of boxes, its coordinate tables on the device
    TmaOperand tmaA;
    const int32_t *d_tma_coord_m = nullptr, *d_tma_coord_k = nullptr, *d_tma_coord_h = nullptr;
    // short-K streaming kernel: piece orders of the operand tiles; how many consecutive m are contiguous in D
    // ([0], [1]: the plan's A as the kernel's M side / N side; [2], [3]: the plan's B likewise)
    std::vector<uint32_t> skinny_order[4];
    const uint32_t *d_skinny_order[4] = {nullptr, nullptr, nullptr, nullptr};
    int64_t skinny_run_m = 1;
    bool skinny_regular = false;
    bool skinny_d_regular[2] = {false, false};     // D's rows (m) / columns (n) regular
    size_t workspace_bytes = 0;
    size_t workspace_floor = 0;   // what the operation needs at least (without the real form of complex64, which is then not used)
    int32_t grid[3] = {0, 0, 0};
    // Case 4: inputs with isolated labels are first summed into the front of the workspace
    // (A' at offset 0, B' behind it), split-K partial sums follow at `partials_offset`
    bool pre_reduce = true;
    uint32_t poll_limit = kWaitPollLimit;   // BTC_ATTR_POLL_LIMIT
    IsolatedSum sumA, sumB;
    size_t sumB_offset = 0, partials_offset = 0;
    // memory spans of the caller's tensors in elements (the plan may describe A' and B' instead)
    int64_t spanA_lo = 0, spanA_hi = 0, spanB_lo = 0, spanB_hi = 0, spanD_lo = 0, spanD_hi = 0;
    struct HostPipeline *host = nullptr;   // built by the first btc_execute_host
    // complex64 on the fp32 tensor-core path (complex_expand_kernel.cuh): the smaller input X is expanded
    // into the front of the workspace, then `real_inner`, an fp32 contraction over the real views, runs.
    // Used when that operation lands on a tcgen05 kernel; beta must be real and C not conjugated at execute.
    btc_contraction_s *real_inner = nullptr;
    bool real_expand_A = true;              // X is the caller's A (else B)
    ComplexExpandParams real_expand;        // loop dimensions of X in X'' order (pointers and scalars filled at execute)
    size_t real_x_bytes = 0;                // bytes of X'' (rounded up to 256)
    // One real and one complex input (mixed element types): with the complex tensors read as real tensors
    // with one more mode (the part, a free label of the complex input and of D) the operation is an
    // ordinary real contraction, `real_inner` with real_view_only set: nothing is expanded.
    bool real_view_only = false;
};

// Host-buffer execution in slabs (btc_execute_host): the larger input is cut along the label with its largest
// stride, slab i + 1 is copied to the device while slab i is contracted.
struct HostPipeline {
    bool tried = false, usable = false;
    bool slab_is_A = true;                 // which caller-side input is cut
    int64_t extent = 0, slab = 0;          // extent of the cut label, slab length
    int idxX = -1, idxY = -1, idxD = -1;   // position of the label in the cut input, the other input, D (-1: absent)
    int64_t strideX = 0, strideY = 0, strideD = 0;
    btc_contraction_s *sub[2] = {nullptr, nullptr};   // operation for a full slab / for the remainder
    int64_t sub_lo[2] = {0, 0}, sub_hi[2] = {0, 0};   // span of a slab of the cut input (elements, relative to its first element)
    char *bufX[2] = {nullptr, nullptr}, *bufY = nullptr, *bufD = nullptr, *bufC = nullptr, *ws = nullptr;
    size_t bytesX = 0, bytesY = 0, bytesD = 0, bytesC = 0, bytesW = 0;
    cudaStream_t copy_stream = nullptr;
    cudaEvent_t loaded[2] = {nullptr, nullptr}, consumed[2] = {nullptr, nullptr};
};

struct btc_elementwise_s {
    btc_handle_s handle;
    ElementwiseRequest req;
    ElementwisePlan plan;
    double alpha[2] = {1.0, 0.0}, beta[2] = {0.0, 0.0};
    int32_t last_kernel = 0;      // what the last execute launched: 1 direct, 2 transposing, 3 vector
};

namespace {

void free_host_pipeline(btc_contraction_s *op);

// ---- tiled kernel variants -------------------------------------------------------------------
using F64Big = F64Tile<false, 128, 128, 2, 4, 4, 1>;
using F64Small = F64Tile<false, 64, 64, 2, 4, 4, 2>;             // 8 consumer warps: two per scheduler
using F64Big16 = F64Tile<false, 128, 128, 2, 4, 4, 1, true>;   // m16n8k16 MMAs
using F64Big3 = F64Tile<false, 128, 128, 2, 4, 3, 1>;           // 3 stages
using F64BigT = F64Tile<false, 128, 128, 4, 2, 4, 1>;           // warp tile 32 x 64
using C64Big = F64Tile<true, 128, 64, 2, 4, 4, 1>;
using C64Small = F64Tile<true, 64, 32, 2, 4, 4, 2>;
using C64Big16 = F64Tile<true, 128, 64, 2, 4, 4, 1, true>;     // m16n8k16 MMAs

using F32Big = F32Tile<128, 128, 16, 2, 4, 5, 1, false>;
using F32Small = F32Tile<64, 64, 16, 2, 2, 5, 2, false>;
using F32Wide = F32Tile<256, 96, 16, 4, 2, 5, 1, false>;       // N = 96 fills the tile exactly
using F32BigP = F32Tile<128, 128, 16, 2, 4, 5, 1, true>;
using F32WideP = F32Tile<256, 96, 16, 4, 2, 5, 1, true>;
using F32Big32 = F32Tile<128, 128, 32, 2, 4, 3, 1, false>;
using F32Tc = TF32Tile<false, 128, 128, 2, 4, 4, 1>;             // 3xTF32 on the tensor cores
using F32TcSmall = TF32Tile<false, 64, 64, 2, 4, 4, 2>;
using F32TcTiny = TF32Tile<false, 64, 64, 2, 4, 2, 3>;            // two stages, three CTAs per SM: short-K, low-intensity problems
using C32Tc = TF32Tile<true, 128, 64, 2, 4, 4, 1>;
using C32TcSmall = TF32Tile<true, 64, 32, 2, 4, 4, 2>;
using F32TcWide = TF32Tile<false, 256, 96, 4, 2, 4, 1>;          // N = 96 fills the tile exactly
using F32TcMid = TF32Tile<false, 128, 96, 2, 4, 4, 1>;
using F32Umma96 = UmmaTile<96, 4, 2>;
using F32Umma96T = UmmaTile<96, 5, 2, true>;                       // M-side operand through tensor memory
using F32Umma128T = UmmaTile<128, 4, 2, true>;
using F32Umma96T2 = UmmaTile<96, 5, 2, true, 2>;                   // two converter groups take the stages in turn
using F32Umma128T2 = UmmaTile<128, 4, 2, true, 2>;                              // tcgen05 + tensor memory, 3xTF32
using F32Umma128 = UmmaTile<128, 4, 2>;
using F32Umma256 = UmmaTile<256, 3, 1>;
// M side fetched by bulk tensor copies (one box per stage), stages of 24 or 32 k
using F32Umma96B24 = UmmaTile<96, 7, 2, true, 1, 24, true>;
using F32Umma96B32 = UmmaTile<96, 5, 2, true, 1, 32, true>;
using F32Umma128B32 = UmmaTile<128, 4, 2, true, 1, 32, true>;
using F32Umma128B24 = UmmaTile<128, 5, 2, true, 1, 24, true>;
using F32Umma96B24x2 = UmmaTile<96, 3, 2, true, 1, 24, true, 2>;   // two sub-stages of 24 k per hand-off
constexpr int kNumF32Variants = 24;
constexpr int kFirstUmmaVariant = 10;
constexpr int kFirstBulkVariant = 17;     // 17..21: bulk tensor copies; fall back to 13 / 14 (same tiles) at execute
constexpr int SKINNY_LINES = 256;         // 128-byte lines of a 32 KiB operand tile
constexpr int kSkinnyVariant = 23;        // short-K streaming kernel (tcgen05); falls back to 6 (same tiles) at execute
// fp32 variants whose CTAs are persistent and keep all of K (no split-K)
inline bool f32_persistent(int variant) { return (variant >= kFirstUmmaVariant && variant <= 21) || variant == kSkinnyVariant; }

struct VariantInfo {
    int bm, bn, bk, threads, acc;
    size_t smem, acc_bytes;
};
// `threads` counts the consumer threads: they own the accumulators (split-K scratch layout)
template <typename T> VariantInfo info_of(size_t acc_bytes)
{
    return {T::BM, T::BN, T::BK, T::CONSUMER_THREADS, T::ACC, T::SMEM_BYTES, acc_bytes};
}

bool tiled_supported(btc_dtype_t) { return true; }

VariantInfo variant_info(btc_dtype_t t, int variant)
{
    if (t == BTC_F64) {
        switch (variant) {
        case 0: return info_of<F64Big>(8);
        case 1: return info_of<F64Small>(8);
        case 2: return info_of<F64Big16>(8);
        case 3: return info_of<F64Big3>(8);
        default: return info_of<F64BigT>(8);
        }
    }
    if (t == BTC_F32) {
        switch (variant) {
        case 0: return info_of<F32Big>(4);
        case 1: return info_of<F32Small>(4);
        case 2: return info_of<F32Wide>(4);
        case 3: return info_of<F32BigP>(4);
        case 4: return info_of<F32WideP>(4);
        case 5: return info_of<F32Big32>(4);
        case 6: return info_of<F32Tc>(4);
        case 7: return info_of<F32TcSmall>(4);
        case 8: return info_of<F32TcWide>(4);
        case 9: return info_of<F32TcMid>(4);
        case 10: return {128, 96, 32, 256, 0, F32Umma96::SMEM_BYTES, 4};
        case 11: return {128, 128, 32, 256, 0, F32Umma128::SMEM_BYTES, 4};
        case 12: return {128, 256, 32, 256, 0, F32Umma256::SMEM_BYTES, 4};
        case 13: return {128, 96, 32, 256, 0, F32Umma96T::SMEM_BYTES, 4};
        case 14: return {128, 128, 32, 256, 0, F32Umma128T::SMEM_BYTES, 4};
        case 15: return {128, 96, 32, 256, 0, F32Umma96T2::SMEM_BYTES, 4};
        case 17: return {128, 96, 24, 256, 0, F32Umma96B24::SMEM_BYTES, 4};
        case 18: return {128, 96, 32, 256, 0, F32Umma96B32::SMEM_BYTES, 4};
        case 19: return {128, 128, 32, 256, 0, F32Umma128B32::SMEM_BYTES, 4};
        case 20: return {128, 128, 24, 256, 0, F32Umma128B24::SMEM_BYTES, 4};
        case 21: return {128, 96, 24, 256, 0, F32Umma96B24x2::SMEM_BYTES, 4};
        case 22: return info_of<F32TcTiny>(4);
        case 23: return {128, 128, 64, 256, 0, 0, 4};
        default: return {128, 128, 32, 256, 0, F32Umma128T2::SMEM_BYTES, 4};
        }
    }
    if (t == BTC_C32) return variant == 0 ? info_of<C32Tc>(4) : info_of<C32TcSmall>(4);
    return variant == 0 ? info_of<C64Big>(8) : (variant == 1 ? info_of<C64Small>(8) : info_of<C64Big16>(8));
}

// (racing first calls on one device both set the attribute: harmless; the flags are atomics so that
// host threads may execute concurrently)
template <typename K>
cudaError_t set_smem_once(K kernel, size_t bytes, std::atomic<bool> *configured)
{
    int dev = 0;
    cudaGetDevice(&dev);
    if (dev >= 0 && dev < 64 && !configured[dev].load(std::memory_order_relaxed)) {
        cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, int(bytes));
        if (e != cudaSuccess) return e;
        configured[dev].store(true, std::memory_order_relaxed);
    }
    return cudaSuccess;
}

template <typename T>
cudaError_t launch_tiled(const TiledParams &p, int64_t ctas, int64_t reduce_ctas, cudaStream_t st)
{
    static std::atomic<bool> configured[64] = {};
    cudaError_t e = set_smem_once(tiled_f64_kernel<T>, T::SMEM_BYTES, configured);
    if (e != cudaSuccess) return e;
    if (p.cluster_split) {
        // the k slices of a tile as one thread-block cluster: they add up through distributed shared memory
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(unsigned(ctas)); cfg.blockDim = dim3(T::THREADS);
        cfg.dynamicSmemBytes = T::SMEM_BYTES; cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = unsigned(p.split_k); attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, tiled_f64_kernel<T>, p);
    }
    tiled_f64_kernel<T><<<unsigned(ctas), T::THREADS, T::SMEM_BYTES, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (p.split_k > 1) {
        splitk_reduce_kernel<double, T::W><<<unsigned(reduce_ctas), 256, 0, st>>>(p);
        e = cudaGetLastError();
    }
    return e;
}

template <typename T>
cudaError_t launch_tiled_tf32(const TiledParams &p, int64_t ctas, int64_t reduce_ctas, cudaStream_t st)
{
    static std::atomic<bool> configured[64] = {};
    cudaError_t e = set_smem_once(tiled_tf32x3_kernel<T>, T::SMEM_BYTES, configured);
    if (e != cudaSuccess) return e;
    tiled_tf32x3_kernel<T><<<unsigned(ctas), T::THREADS, T::SMEM_BYTES, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (p.split_k > 1) {
        splitk_reduce_kernel<float, T::W><<<unsigned(reduce_ctas), 256, 0, st>>>(p);
        e = cudaGetLastError();
    }
    return e;
}

template <typename T>
cudaError_t launch_umma(const TiledParams &p, int64_t ctas, cudaStream_t st, const CUtensorMap *mapA = nullptr)
{
    static std::atomic<bool> configured[64] = {};
    cudaError_t e = set_smem_once(tiled_umma_tf32x3_kernel<T>, T::SMEM_BYTES, configured);
    if (e != cudaSuccess) return e;
    static const CUtensorMap none = {};
    tiled_umma_tf32x3_kernel<T><<<unsigned(ctas), T::THREADS, T::SMEM_BYTES, st>>>(p, mapA ? *mapA : none);
    return cudaGetLastError();
}

// Tensor map of the M-side operand for the bulk-copy variants: fp32 elements, the planner's
// dimensions and box, zero fill outside the tensor, 128-byte swizzle when a box row is 128 bytes
// of k.  The encoder is a driver entry point looked up once through the runtime (no link-time
// dependency on the driver library).  False when the driver declines the description.
bool encode_tma_operand(const TmaOperand &t, const void *base, CUtensorMap *out)
{
    using Encode = CUresult (*)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static Encode encode = [] {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
            cudaGetLastError();
            fn = nullptr;
        }
        return reinterpret_cast<Encode>(fn);
    }();
    if (!encode || !t.ok) return false;
    cuuint64_t dim[5], stride[4];
    cuuint32_t box[5], estr[5] = {1, 1, 1, 1, 1};
    for (int d = 0; d < 5; ++d) { dim[d] = t.dim[d]; box[d] = t.box[d]; }
    for (int d = 1; d < 5; ++d) stride[d - 1] = t.stride[d] * 4;
    const bool swz = t.k_major && t.box[0] == 32;
    return encode(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 5, const_cast<void *>(base), dim, stride, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, swz ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <typename T, bool AK, bool BK_>
cudaError_t launch_tiled_f32_o(const TiledParams &p, int64_t ctas, int64_t reduce_ctas, cudaStream_t st)
{
    static std::atomic<bool> configured[64] = {};
    cudaError_t e = set_smem_once(tiled_f32_kernel<T, AK, BK_>, T::SMEM_BYTES, configured);
    if (e != cudaSuccess) return e;
    tiled_f32_kernel<T, AK, BK_><<<unsigned(ctas), T::THREADS, T::SMEM_BYTES, st>>>(p);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    if (p.split_k > 1) {
        splitk_reduce_kernel<float, 1><<<unsigned(reduce_ctas), 256, 0, st>>>(p);
        e = cudaGetLastError();
    }
    return e;
}

// the shared-memory orientation of each operand is a compile-time property of the fp32 kernel
template <typename T>
cudaError_t launch_tiled_f32(const TiledParams &p, int64_t ctas, int64_t reduce_ctas, cudaStream_t st)
{
    if (p.dirA) return p.dirB ? launch_tiled_f32_o<T, true, true>(p, ctas, reduce_ctas, st)
                              : launch_tiled_f32_o<T, true, false>(p, ctas, reduce_ctas, st);
    return p.dirB ? launch_tiled_f32_o<T, false, true>(p, ctas, reduce_ctas, st)
                  : launch_tiled_f32_o<T, false, false>(p, ctas, reduce_ctas, st);
}

void to_double2(btc_dtype_t t, const void *src, double out[2])
{
    switch (t) {
    case BTC_F32: out[0] = *static_cast<const float *>(src); out[1] = 0; break;
    case BTC_F64: out[0] = *static_cast<const double *>(src); out[1] = 0; break;
    case BTC_C32: out[0] = static_cast<const float *>(src)[0]; out[1] = static_cast<const float *>(src)[1]; break;
    case BTC_C64: out[0] = static_cast<const double *>(src)[0]; out[1] = static_cast<const double *>(src)[1]; break;
    }
}

void free_tables(btc_contraction_s *op)
{
    if (op->d_tables) cudaFree(op->d_tables);
    op->d_tables = nullptr;
    op->d_error = nullptr;
}

// Choose tile variant, raster order and split-K for a tiled plan; upload the offset tables.
int finish_plan(btc_contraction_s *op)
{
    Plan &pl = op->plan;
    free_tables(op);
    op->workspace_bytes = 0;
    if (pl.kernel == BTC_KERNEL_TILED && !tiled_supported(pl.dtype)) {
        if (op->req.force_kernel == BTC_KERNEL_TILED) return BTC_ERR_NOT_SUPPORTED;
        pl.kernel = BTC_KERNEL_GENERIC;
    }
    if (pl.kernel == BTC_KERNEL_GENERIC) {
        if (pl.batch.size() + pl.m.size() + pl.n.size() > size_t(kGenericMaxD) || pl.k.size() > size_t(kGenericMaxK))
            return BTC_ERR_NOT_SUPPORTED;
        const double total = double(pl.Bt) * double(pl.M) * double(pl.N);
        const bool warp_per_elem = total < 4096.0 * 8 && pl.K >= 64;
        const int64_t groups = pl.Bt * pl.M * pl.N;
        const int64_t threads = warp_per_elem ? groups * 32 : groups;
        int64_t blocks = (threads + 255) / 256;
        const int64_t cap = int64_t(op->handle.sm_count) * 32;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        op->grid[0] = int32_t(blocks); op->grid[1] = warp_per_elem ? 32 : 1; op->grid[2] = 1;
        pl.tile = TileConfig();
        pl.split_k = 1;
        if (op->handle.device >= 0) {            // no tables, only the device error word
            if (cudaMalloc(reinterpret_cast<void **>(&op->d_tables), 256) != cudaSuccess) { cudaGetLastError(); op->d_tables = nullptr; return BTC_ERR_OUT_OF_MEMORY; }
            if (cudaMemset(op->d_tables, 0, 256) != cudaSuccess) { cudaGetLastError(); return BTC_ERR_CUDA; }
            op->d_error = reinterpret_cast<int32_t *>(op->d_tables);
        }
        return BTC_SUCCESS;
    }

    const int sms = op->handle.sm_count;
    auto tiles_for = [&](const VariantInfo &v) {
        return ((pl.M + v.bm - 1) / v.bm) * ((pl.N + v.bn - 1) / v.bn) * pl.Bt;
    };
    // tiles in flight at a time when the operation runs over a pointer array (BTC_ATTR_BATCH_HINT):
    // what tile choice and split-K are judged by; grid and workspace stay those of one entry
    const int64_t hint = op->req.batch_hint > 1 ? op->req.batch_hint : 1;
    // Candidate tile variants of the element type (fp32: the 3xTF32 tensor-core variants, mma.sync
    // or tcgen05; the strict-fp32 FFMA variants 0-5 are selected with BTC_ATTR_VARIANT only).  Score = fraction of
    // the padded tiles that is real work x fraction of the last wave that is filled x a mild
    // preference for larger tiles (more flops per byte moved through shared memory).
    int variant = 0;
    {
        struct Cand { int id; double weight; };
        // The tcgen05 variants (10-16; candidates: 128x256 with both operands in shared memory,
        // 128x128 and 128x96 with the M side through tensor memory) keep all of K in one CTA and have a longer prologue: they
        // enter only when there is enough work to fill the SMs without split-K; their weights
        // reflect measured throughput relative to the mma.sync variants.
        const double flops = 2.0 * double(pl.M) * double(pl.N) * double(pl.K) * double(pl.Bt);
        // (measured against the mma.sync variants with their split-K: ahead from about 0.6 GFLOP on when 128 x 128
        // tiles fill at least 64 SMs -- 1024 x 1024 x 512: 25 against 31 us, 4096 x 512 x 256: 19 against 47 us --
        // and on a par at 512^3)
        const double tiles128 = double((pl.M + 127) / 128) * double((pl.N + 127) / 128) * double(pl.Bt) * double(hint);
        const bool umma_ok = pl.dtype == BTC_F32 && pl.K >= 64 &&
                             (flops * double(hint) >= 2e9 || (flops * double(hint) >= 0.6e9 && tiles128 >= 64.0));
        // 17-20 fetch the M side with bulk tensor copies; they enter when that operand is a tensor of boxes
        TmaOperand probe;
        const bool box24 = umma_ok && make_tma_operand(pl, 128, 24, probe), box32 = umma_ok && make_tma_operand(pl, 128, 32, probe);
        // (weights from the batched permuted workload: 21, two sub-stages of 24 k per hand-off, is 2 % ahead of
        // the gathering variant 13, the single-sub-stage ones 17-20 a little behind their twins 13 / 14)
        // (measured on 4096 x 4096 x 2048 fp32 in three operand layouts: 19: 222-224 TFLOP/s, 14: 206-214, 16: 188-196,
        // 11: 182-185, 12: 152-154; the 128 x 256 tile with both operands in shared memory stays behind)
        const Cand f32c[] = {{6, 1.0}, {8, 1.0}, {9, 0.93}, {7, 0.75}, {12, 1.7}, {14, 2.3}, {13, 2.0},
                             {box24 ? 17 : 13, 1.85}, {box32 ? 18 : 13, 1.95}, {box32 ? 19 : 14, box32 ? 2.45 : 2.3}, {box24 ? 20 : 14, 2.1},
                             {box24 ? 21 : 13, 2.04}};
        const Cand f32strict[] = {{0, 1.0}, {2, 1.0}, {1, 0.75}};   // FFMA kernels: 128x128, 256x96, 64x64
        const Cand f64c[] = {{2, 1.0}, {1, 0.75}};       // big tile: the m16n8k16 variant
        const Cand c64c[] = {{2, 1.0}, {1, 0.75}};       // complex128: big tile on m16n8k16 as well
        const Cand other[] = {{0, 1.0}, {1, 0.75}};
        const bool strict = pl.dtype == BTC_F32 && op->req.strict_fp32 != 0;
        const Cand *cands = strict ? f32strict : (pl.dtype == BTC_F32 ? f32c : (pl.dtype == BTC_F64 ? f64c : (pl.dtype == BTC_C64 ? c64c : other)));
        const int ncand = strict ? 3 : (pl.dtype == BTC_F32 ? (umma_ok ? 12 : 4) : 2);
        double best = -1.0;
        for (int c = 0; c < ncand; ++c) {
            const VariantInfo vi = variant_info(pl.dtype, cands[c].id);
            const double tiles = double(tiles_for(vi)) * double(hint);
            const double ctas_per_sm = vi.bm * vi.bn <= 64 * 64 ? 2.0 : 1.0;
            const double slots = sms * ctas_per_sm;
            const double util = double(pl.M) * double(pl.N) * double(pl.Bt) * double(hint) / (tiles * vi.bm * vi.bn);
            const double waves = std::ceil(tiles / slots);
            const double wave_eff = tiles / (waves * slots);
            const double score = util * wave_eff * cands[c].weight;
            if (score > best) { best = score; variant = cands[c].id; }
        }
    }
    // fp32 with a short contracted extent (all of K in one shared-memory tile): the streaming kernel,
    // when both operands can be fetched in 16-byte pieces and there are enough 128 x 128 tiles to
    // occupy a good part of the machine
    const bool skinny_fits = pl.dtype == BTC_F32 && op->req.strict_fp32 == 0 && pl.K <= kSkinnyMaxK && pl.vecA == 4 && pl.vecB == 4;
    if (skinny_fits && ((pl.M + 127) / 128) * ((pl.N + 127) / 128) * pl.Bt * hint >= 32) variant = kSkinnyVariant;
    // at most four contracted indices (outer products, Hadamard products, a scalar operand): the streaming kernel
    const bool stream_fits = pl.K <= kStreamMaxContracted;
    if (stream_fits) variant = kStreamVariant;
    if (op->req.force_variant == kStreamVariant) {
        if (!stream_fits) return BTC_ERR_NOT_SUPPORTED;
    } else if (op->req.force_variant >= 0) {
        const int count = pl.dtype == BTC_F32 ? kNumF32Variants : (pl.dtype == BTC_F64 ? 5 : (pl.dtype == BTC_C64 ? 3 : 2));
        if (op->req.force_variant >= count) return BTC_ERR_INVALID_ARGUMENT;
        variant = op->req.force_variant;
        if (pl.dtype == BTC_F32 && variant == kSkinnyVariant && !skinny_fits) variant = 6;   // the mma.sync twin (same tiles)
    }
    op->tmaA = TmaOperand();
    if (pl.dtype == BTC_F32 && variant >= kFirstBulkVariant && variant <= 21) {
        // a forced bulk-copy variant whose M-side operand is no tensor of boxes: the gathering twin
        const VariantInfo bv = variant_info(pl.dtype, variant);
        if (!make_tma_operand(pl, bv.bm, bv.bk, op->tmaA)) variant = (variant <= 18 || variant == 21) ? 13 : 14;
    }
    if (variant == kStreamVariant) {
        // no tiles: one thread per 16 bytes of D, grid-stride
        pl.tile = TileConfig();
        pl.tile.variant = variant;
        pl.split_k = 1;
        op->tiles_m = op->tiles_n = 0;
        const int64_t vectors = (pl.M * pl.N * pl.Bt + 3) / 4;
        int64_t blocks = (vectors + 255) / 256;
        const int64_t cap = int64_t(sms) * 32;
        op->grid[0] = int32_t(blocks < 1 ? 1 : (blocks > cap ? cap : blocks)); op->grid[1] = op->grid[2] = 1;
    }
    const VariantInfo v = variant == kStreamVariant ? VariantInfo{1, 1, 1, 0, 0, 0, 0} : variant_info(pl.dtype, variant);
    if (variant != kStreamVariant) {
    pl.tile.bm = v.bm; pl.tile.bn = v.bn; pl.tile.bk = v.bk; pl.tile.threads = v.threads;
    pl.tile.stages = 0; pl.tile.variant = variant;
    op->tiles_m = int32_t((pl.M + v.bm - 1) / v.bm);
    op->tiles_n = int32_t((pl.N + v.bn - 1) / v.bn);
    op->raster_n_fast = op->tiles_n <= op->tiles_m ? 1 : 0;
    const int64_t tiles = tiles_for(v);
    const int64_t k_tiles = (pl.K + v.bk - 1) / v.bk;
    int64_t split = 1;
    const bool umma = pl.dtype == BTC_F32 && f32_persistent(variant);   // these keep all of K in one CTA
    if (umma) {
        split = 1;
    } else if (op->req.force_split_k > 0) {
        split = op->req.force_split_k;
    } else if (tiles * hint < sms) {
        split = (2 * int64_t(sms)) / (tiles * hint);
        const int64_t max_split = k_tiles / 2;   // at least two K tiles per slice
        if (split > max_split) split = max_split;
    } else {
        // A few waves with a poorly filled last one: slicing K by 2-4 makes the CTAs shorter and the
        // last wave fuller.  Cost model in units of one unsplit tile: waves / slices, plus the
        // partial images' round trip through memory (about 50 elements' worth of work per slice).
        const double slots = double(sms) * (v.bm * v.bn <= 64 * 64 ? 2.0 : 1.0);
        double best = std::ceil(double(tiles * hint) / slots);
        for (int64_t sl = 2; sl <= 4 && k_tiles / sl >= 16; ++sl) {
            const double t = std::ceil(double(tiles * hint * sl) / slots) / double(sl) * (1.0 + 50.0 * double(sl) / double(pl.K));
            if (t < 0.97 * best) { best = t; split = sl; }
        }
    }
    if (split > k_tiles) split = k_tiles;
    if (split < 1) split = 1;
    int64_t kt_per = (k_tiles + split - 1) / split;
    split = (k_tiles + kt_per - 1) / kt_per;     // no empty slices
    pl.split_k = int32_t(split);
    op->k_per_split = kt_per * v.bk;
    if (tiles * split > 0x7fffffffLL) return BTC_ERR_NOT_SUPPORTED;
    op->grid[0] = int32_t(tiles * split); op->grid[1] = 1; op->grid[2] = 1;
    if (umma && op->grid[0] > sms) op->grid[0] = int32_t(sms);   // persistent CTAs walk the tile list
    if (split > 1)
        op->workspace_bytes = size_t(tiles) * size_t(split) * size_t(v.threads) * size_t(v.acc) * v.acc_bytes;
    }   // tiled variants

    for (auto &o : op->skinny_order) o.clear();
    if (pl.dtype == BTC_F32 && variant == kSkinnyVariant) {
        // Piece orders.  An operand tile (128 rows x K padded to a multiple of 8) is fetched in 16-byte
        // pieces, 32 per warp instruction.  Such a copy runs at full speed when its 32 destinations fill
        // whole 128-byte lines of shared memory and its sources few lines of global memory, so the
        // pieces are grouped by the shared-memory line they land in (which depends on the side of the
        // kernel the operand plays), pieces of a line in position order, and the lines sorted by the
        // address of their first piece in the tensor.  Every tile uses the order computed for the first:
        // any order is correct, this one is fast whenever tiles are laid out alike.
        const int kp = int((pl.K + 7) / 8 * 8);
        auto operand_order = [&](const std::vector<int64_t> &row_off, const std::vector<int64_t> &k_off, int64_t rows, LoadDir dir, bool n_side) {
            struct Piece { int64_t addr; unsigned dst; uint16_t e; };
            std::vector<Piece> v;
            const int d = dir == LoadDir::ALONG_FREE ? 0 : 1;
            for (int e = 0; e < 32 * kp; ++e) {
                int row, k;
                const unsigned dst = n_side ? skinny_b_pos(d, unsigned(e), row, k) : skinny_a_pos(d, unsigned(e), row, k);
                v.push_back({(row < rows && k < pl.K) ? row_off[size_t(row)] + k_off[size_t(k)] : INT64_MAX, dst, uint16_t(e)});
            }
            std::vector<int64_t> first(size_t(SKINNY_LINES), INT64_MAX);     // smallest address of each line
            for (auto &x : v) first[x.dst >> 7] = std::min(first[x.dst >> 7], x.addr);
            std::stable_sort(v.begin(), v.end(), [&](const Piece &a, const Piece &b) {
                const unsigned la = a.dst >> 7, lb = b.dst >> 7;
                if (la == lb) return a.dst < b.dst;
                return first[la] != first[lb] ? first[la] < first[lb] : la < lb;
            });
            // per piece, in that order: bits 0-10 the piece, bit 11 its k < K, bits 12-31 (signed) its offset
            // relative to the tile's first row in units of four elements (used for regular operands only)
            std::vector<uint32_t> out;
            for (auto &x : v) {
                int row, k;
                if (n_side) skinny_b_pos(d, unsigned(x.e), row, k); else skinny_a_pos(d, unsigned(x.e), row, k);
                const int64_t rel = (row < rows && k < pl.K) ? row_off[size_t(row)] - row_off[0] + k_off[size_t(k)] : 0;
                out.push_back(uint32_t(x.e) | (uint32_t(k < pl.K) << 11) | (uint32_t(int32_t(rel / 4)) << 12));
            }
            return out;
        };
        op->skinny_order[0] = operand_order(pl.offA_m, pl.offA_k, pl.M, pl.dirA, false);
        op->skinny_order[1] = operand_order(pl.offA_m, pl.offA_k, pl.M, pl.dirA, true);
        op->skinny_order[2] = operand_order(pl.offB_n, pl.offB_k, pl.N, pl.dirB, false);
        op->skinny_order[3] = operand_order(pl.offB_n, pl.offB_k, pl.N, pl.dirB, true);
        // regular operand: rows m0 + r of every tile lie relative to row m0 as rows r of tile 0 relative to row 0
        auto regular = [&](const std::vector<int64_t> &row_off, const std::vector<int64_t> &k_off) {
            const int64_t n = int64_t(row_off.size());
            int64_t lo = 0, hi = 0;
            for (int64_t r = 0; r < n; ++r) {
                const int64_t rel = row_off[size_t(r)] - row_off[size_t(r - r % 128)];
                if (rel != row_off[size_t(r % 128)] - row_off[0]) return false;
                lo = std::min(lo, rel); hi = std::max(hi, rel);
            }
            int64_t klo = 0, khi = 0;
            for (int64_t k = 0; k < int64_t(k_off.size()); ++k) { klo = std::min(klo, k_off[size_t(k)]); khi = std::max(khi, k_off[size_t(k)]); }
            // (offsets inside a tile are kept in 20 bits, in units of four elements)
            return hi + khi < (int64_t(1) << 20) && lo + klo > -(int64_t(1) << 20);
        };
        op->skinny_regular = regular(pl.offA_m, pl.offA_k) && regular(pl.offB_n, pl.offB_k);
        const std::vector<int64_t> none(1, 0);
        op->skinny_d_regular[0] = regular(pl.offD_m, none);
        op->skinny_d_regular[1] = regular(pl.offD_n, none);
        // consecutive m that are consecutive elements of D
        op->skinny_run_m = 1;
        for (auto &md : pl.m) {
            if (md.sD != op->skinny_run_m) break;
            op->skinny_run_m *= md.extent;
        }
    }

    if (op->handle.device >= 0) {
        const std::vector<int64_t> *tabs[9] = {&pl.offA_m, &pl.offD_m, &pl.offB_n, &pl.offD_n, &pl.offA_k,
                                               &pl.offB_k, &pl.offA_h, &pl.offB_h, &pl.offD_h};
        const int64_t **dst[9] = {&op->d_offA_m, &op->d_offD_m, &op->d_offB_n, &op->d_offD_n, &op->d_offA_k,
                                  &op->d_offB_k, &op->d_offA_h, &op->d_offB_h, &op->d_offD_h};
        size_t total = 0;
        for (auto *t : tabs) total += (t->size() + 31) / 32 * 32;   // keep every table 256-byte aligned
        const size_t error_at = total;
        total += 32;                                                  // the error word, zeroed
        // coordinate tables of the bulk-copy variants (int32), packed behind the error word
        const std::vector<int32_t> *ctabs[3] = {&op->tmaA.coordM, &op->tmaA.coordK, &op->tmaA.coordH};
        size_t cstart[3];
        for (int i = 0; i < 3; ++i) {
            cstart[i] = total;
            total += (ctabs[i]->size() + 63) / 64 * 32;
        }
        // piece orders of the short-K streaming kernel, as raw bytes
        const void *blob[4];
        size_t blob_bytes[4], bstart[4];
        for (int i = 0; i < 4; ++i) {
            blob[i] = op->skinny_order[i].data();
            blob_bytes[i] = op->skinny_order[i].size() * 4;
            bstart[i] = total;
            total += (blob_bytes[i] + 255) / 256 * 32;
        }
        std::vector<int64_t> host(total, 0);
        for (int i = 0; i < 3; ++i)
            if (!ctabs[i]->empty()) std::memcpy(host.data() + cstart[i], ctabs[i]->data(), ctabs[i]->size() * sizeof(int32_t));
        for (int i = 0; i < 4; ++i)
            if (blob_bytes[i]) std::memcpy(host.data() + bstart[i], blob[i], blob_bytes[i]);
        size_t pos = 0, starts[9];
        for (int i = 0; i < 9; ++i) {
            starts[i] = pos;
            std::memcpy(host.data() + pos, tabs[i]->data(), tabs[i]->size() * sizeof(int64_t));
            pos += (tabs[i]->size() + 31) / 32 * 32;
        }
        if (cudaMalloc(reinterpret_cast<void **>(&op->d_tables), total * sizeof(int64_t)) != cudaSuccess) {
            cudaGetLastError();
            op->d_tables = nullptr;
            return BTC_ERR_OUT_OF_MEMORY;
        }
        if (cudaMemcpy(op->d_tables, host.data(), total * sizeof(int64_t), cudaMemcpyHostToDevice) != cudaSuccess) {
            cudaGetLastError();
            return BTC_ERR_CUDA;
        }
        for (int i = 0; i < 9; ++i) *dst[i] = op->d_tables + starts[i];
        op->d_error = reinterpret_cast<int32_t *>(op->d_tables + error_at);
        op->d_tma_coord_m = reinterpret_cast<const int32_t *>(op->d_tables + cstart[0]);
        op->d_tma_coord_k = reinterpret_cast<const int32_t *>(op->d_tables + cstart[1]);
        op->d_tma_coord_h = reinterpret_cast<const int32_t *>(op->d_tables + cstart[2]);
        for (int i = 0; i < 4; ++i) op->d_skinny_order[i] = reinterpret_cast<const uint32_t *>(op->d_tables + bstart[i]);
    }
    return BTC_SUCCESS;
}

int replan(btc_contraction_s *op);

void free_real_form(btc_contraction_s *op)
{
    if (op->real_inner) {
        free_tables(op->real_inner);
        delete op->real_inner;
        op->real_inner = nullptr;
    }
    op->real_x_bytes = 0;
    op->real_view_only = false;
}

// Mixed element types, one real and one complex input: D = alpha A B with A real is, part by part, the real
// contraction of A with B read as a real tensor (Eq. (case2) holds for each part).  Needs real scalars and no
// conjugation of the complex tensors at execute; then the tiled kernels of the part type run instead of
// the per-element kernel.
void build_mixed_real_view(btc_contraction_s *op)
{
    const PlanRequest &rq = op->req;
    const Plan &pl = op->plan;
    if (op->handle.device < 0 || !pl.mixed || rq.force_kernel == BTC_KERNEL_GENERIC) return;
    const bool ca = dtype_is_complex(rq.A.dtype), cb = dtype_is_complex(rq.B.dtype);
    if (ca == cb || !dtype_is_complex(rq.D.dtype) || (rq.has_c && rq.C.dtype != rq.D.dtype)) return;
    if ((ca && rq.conjA) || (cb && rq.conjB)) return;
    const btc_dtype_t part = rq.D.dtype == BTC_C32 ? BTC_F32 : BTC_F64;
    int64_t top = 0;
    for (auto *l : {&rq.labelsA, &rq.labelsB, &rq.labelsC, &rq.labelsD}) for (int64_t x : *l) top = std::max(top, x);
    if (top > INT64_MAX - 1) return;
    const int64_t V = top + 1;
    auto real_view = [&](const TensorDesc &t, const std::vector<int64_t> &labels, TensorDesc &out, std::vector<int64_t> &lout) {
        out.dtype = part;
        out.extent.assign(1, 2); out.stride.assign(1, 1); lout.assign(1, V);
        for (size_t i = 0; i < t.extent.size(); ++i) {
            out.extent.push_back(t.extent[i]); out.stride.push_back(2 * t.stride[i]); lout.push_back(labels[i]);
        }
    };
    btc_contraction_s *in = new (std::nothrow) btc_contraction_s;
    if (!in) return;
    in->handle = op->handle;
    in->req = rq;                                    // attributes (precision, hints, forced variants) carry over
    in->req.conjA = in->req.conjB = in->req.conjC = false;
    if (ca) real_view(rq.A, rq.labelsA, in->req.A, in->req.labelsA); else in->req.A.dtype = part;
    if (cb) real_view(rq.B, rq.labelsB, in->req.B, in->req.labelsB); else in->req.B.dtype = part;
    real_view(rq.D, rq.labelsD, in->req.D, in->req.labelsD);
    if (rq.has_c) real_view(rq.C, rq.labelsC, in->req.C, in->req.labelsC);
    in->poll_limit = op->poll_limit;
    in->pre_reduce = op->pre_reduce;
    in->alpha[0] = op->alpha[0]; in->alpha[1] = 0.0; in->beta[0] = op->beta[0]; in->beta[1] = 0.0;
    if (replan(in) != BTC_SUCCESS || in->plan.kernel != BTC_KERNEL_TILED) {
        free_tables(in);
        delete in;
        return;
    }
    op->real_inner = in;
    op->real_view_only = true;
    op->real_x_bytes = 0;
    op->workspace_bytes = std::max(op->workspace_floor, in->workspace_bytes);
}

// complex64 -> fp32: set up the real form of the operation (complex_expand_kernel.cuh) when it is worth
// it, i.e. when the real contraction is planned onto a tcgen05 kernel.  Leaves op->real_inner null otherwise.
void build_real_form(btc_contraction_s *op)
{
    free_real_form(op);
    const PlanRequest &rq = op->req;
    const Plan &pl = op->plan;
    if (op->handle.device < 0 || pl.dtype != BTC_C32 || pl.mixed || pl.has_isolated || pl.kernel != BTC_KERNEL_TILED ||
        rq.strict_fp32 != 0 || rq.force_variant >= 0 || rq.force_split_k != 0)
        return;
    auto count = [](const TensorDesc &t) { int64_t n = 1; for (int64_t e : t.extent) n *= e; return n; };
    auto distinct = [](const std::vector<int64_t> &l) {
        for (size_t i = 0; i < l.size(); ++i)
            for (size_t j = i + 1; j < l.size(); ++j) if (l[i] == l[j]) return false;
        return true;
    };
    const bool expand_A = count(rq.A) <= count(rq.B);
    const TensorDesc &X = expand_A ? rq.A : rq.B, &Y = expand_A ? rq.B : rq.A;
    const std::vector<int64_t> &lX = expand_A ? rq.labelsA : rq.labelsB, &lY = expand_A ? rq.labelsB : rq.labelsA;
    if (!distinct(lX) || X.extent.size() + 2 > size_t(kExpandMaxD)) return;
    auto find = [](const std::vector<int64_t> &l, int64_t x) { for (size_t i = 0; i < l.size(); ++i) if (l[i] == x) return int(i); return -1; };
    // two labels of our own: u (parts of Y, contracted) and v (parts of D)
    int64_t top = 0;
    for (auto *l : {&rq.labelsA, &rq.labelsB, &rq.labelsC, &rq.labelsD}) for (int64_t x : *l) top = std::max(top, x);
    if (top > INT64_MAX - 2) return;
    const int64_t U = top + 1, V = top + 2;
    // X's loop dimensions in the order of X'': contracted ones by |stride in Y|, then the others by |stride in D|
    struct Dim { int64_t label, ext, sx, key; };
    std::vector<Dim> kc, rest;
    for (size_t i = 0; i < lX.size(); ++i) {
        const int iy = find(lY, lX[i]), id = find(rq.labelsD, lX[i]);
        if (id < 0 && iy >= 0) kc.push_back({lX[i], X.extent[i], X.stride[i], std::llabs(Y.stride[size_t(iy)])});
        else if (id >= 0) rest.push_back({lX[i], X.extent[i], X.stride[i], std::llabs(rq.D.stride[size_t(id)])});
        else return;                        // a label of X alone (Case 4): not here
    }
    auto by_key = [](const Dim &a, const Dim &b) { return a.key < b.key; };
    std::stable_sort(kc.begin(), kc.end(), by_key);
    std::stable_sort(rest.begin(), rest.end(), by_key);
    ComplexExpandParams ep;
    std::memset(&ep, 0, sizeof ep);
    ep.total = ep.total_k = 1;
    TensorDesc Xr, Yr, Dr, Cr;
    std::vector<int64_t> lXr, lYr, lDr, lCr;
    Xr.dtype = Yr.dtype = Dr.dtype = Cr.dtype = BTC_F32;
    Xr.extent.push_back(2); Xr.stride.push_back(1); lXr.push_back(U);
    int64_t run = 2;
    for (auto &d : kc) {
        ep.ext[ep.nd] = d.ext; ep.stride[ep.nd] = d.sx; ++ep.nd;
        Xr.extent.push_back(d.ext); Xr.stride.push_back(run); lXr.push_back(d.label);
        run *= d.ext; ep.total_k *= d.ext;
    }
    Xr.extent.push_back(2); Xr.stride.push_back(run); lXr.push_back(V);
    run *= 2;
    for (auto &d : rest) {
        ep.ext[ep.nd] = d.ext; ep.stride[ep.nd] = d.sx; ++ep.nd;
        Xr.extent.push_back(d.ext); Xr.stride.push_back(run); lXr.push_back(d.label);
        run *= d.ext;
    }
    ep.total = run / 4;
    auto real_view = [](const TensorDesc &t, const std::vector<int64_t> &labels, int64_t part, TensorDesc &out, std::vector<int64_t> &lout) {
        out.extent.assign(1, 2); out.stride.assign(1, 1); lout.assign(1, part);
        for (size_t i = 0; i < t.extent.size(); ++i) {
            out.extent.push_back(t.extent[i]); out.stride.push_back(2 * t.stride[i]); lout.push_back(labels[i]);
        }
    };
    real_view(Y, lY, U, Yr, lYr);
    real_view(rq.D, rq.labelsD, V, Dr, lDr);
    if (rq.has_c) real_view(rq.C, rq.labelsC, V, Cr, lCr);
    btc_contraction_s *in = new (std::nothrow) btc_contraction_s;
    if (!in) return;
    in->handle = op->handle;
    in->req.A = expand_A ? Xr : Yr; in->req.labelsA = expand_A ? lXr : lYr;
    in->req.B = expand_A ? Yr : Xr; in->req.labelsB = expand_A ? lYr : lXr;
    in->req.D = Dr; in->req.labelsD = lDr;
    in->req.has_c = rq.has_c;
    if (rq.has_c) { in->req.C = Cr; in->req.labelsC = lCr; }
    in->req.batch_hint = rq.batch_hint;
    in->poll_limit = op->poll_limit;
    in->alpha[0] = 1.0; in->alpha[1] = 0.0; in->beta[0] = op->beta[0]; in->beta[1] = 0.0;
    const bool planned = replan(in) == BTC_SUCCESS && in->plan.kernel == BTC_KERNEL_TILED && in->plan.dtype == BTC_F32 &&
                         f32_persistent(in->plan.tile.variant);
    if (!planned) {
        free_tables(in);
        delete in;
        return;
    }
    op->real_inner = in;
    op->real_expand_A = expand_A;
    op->real_expand = ep;
    op->real_x_bytes = (size_t(ep.total) * 16 + 255) / 256 * 256;
    op->workspace_bytes = std::max(op->workspace_floor, op->real_x_bytes + in->workspace_bytes);
}

int replan(btc_contraction_s *op)
{
    free_real_form(op);
    op->req.sm_count = op->handle.sm_count;
    int rc = make_plan(op->req, op->plan);
    if (rc != BTC_SUCCESS) return rc;
    const Plan &pl = op->plan;
    op->spanA_lo = pl.spanA_lo; op->spanA_hi = pl.spanA_hi; op->spanB_lo = pl.spanB_lo; op->spanB_hi = pl.spanB_hi;
    op->spanD_lo = pl.spanD_lo; op->spanD_hi = pl.spanD_hi;
    op->sumA = op->sumB = IsolatedSum();
    op->sumB_offset = op->partials_offset = 0;
    if (pl.has_isolated && op->pre_reduce && !pl.mixed) {
        // Case 4: plan the contraction of the summed inputs A', B' instead
        PlanRequest inner;
        IsolatedSum sa, sb;
        split_isolated(op->req, inner, sa, sb);
        Plan reduced;
        const bool fits = sa.keep_ext.size() <= size_t(kGenericMaxD) && sa.iso_ext.size() <= size_t(kGenericMaxD) &&
                          sb.keep_ext.size() <= size_t(kGenericMaxD) && sb.iso_ext.size() <= size_t(kGenericMaxD);
        if (fits && make_plan(inner, reduced) == BTC_SUCCESS) {
            op->plan = reduced;
            op->sumA = sa;
            op->sumB = sb;
        }
    }
    rc = finish_plan(op);
    if (rc != BTC_SUCCESS) return rc;
    auto round256 = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t esz = dtype_size(op->plan.dtype);
    const size_t bytesA = op->sumA.active ? round256(size_t(op->sumA.total_keep) * esz) : 0;
    const size_t bytesB = op->sumB.active ? round256(size_t(op->sumB.total_keep) * esz) : 0;
    op->sumB_offset = bytesA;
    op->partials_offset = bytesA + bytesB;
    op->workspace_bytes += op->partials_offset;
    op->workspace_floor = op->workspace_bytes;
    build_real_form(op);
    if (!op->real_inner) build_mixed_real_view(op);
    return BTC_SUCCESS;
}

template <typename R, bool CPLX>
cudaError_t launch_isolated_sum(const IsolatedSum &s, const void *src, void *dst, int sm_count, cudaStream_t st)
{
    IsolatedSumParams p;
    std::memset(&p, 0, sizeof p);
    p.src = src; p.dst = dst;
    p.nk = int32_t(s.keep_ext.size()); p.ni = int32_t(s.iso_ext.size());
    p.total_keep = s.total_keep; p.total_iso = s.total_iso;
    for (int i = 0; i < p.nk; ++i) { p.ext_k[i] = s.keep_ext[size_t(i)]; p.str_k[i] = s.keep_str[size_t(i)]; }
    for (int i = 0; i < p.ni; ++i) { p.ext_i[i] = s.iso_ext[size_t(i)]; p.str_i[i] = s.iso_str[size_t(i)]; }
    // contiguous isolated index of whole 16-byte vectors, kept strides and base aligned alike: lanes share
    // result elements and read vectors
    constexpr int64_t V = 16 / int64_t(sizeof(R) * (CPLX ? 2 : 1));
    bool vec = s.iso_ext.size() == 1 && s.iso_str[0] == 1 && s.iso_ext[0] % V == 0 && reinterpret_cast<uintptr_t>(src) % 16 == 0;
    for (size_t i = 0; vec && i < s.keep_str.size(); ++i) vec = s.keep_str[i] % V == 0;
    if (vec) {
        const int64_t nvec = s.iso_ext[0] / V;
        const int log_l = nvec >= 8 ? 3 : nvec >= 4 ? 2 : nvec >= 2 ? 1 : 0;
        int64_t blocks = ((s.total_keep << log_l) + 255) / 256;
        const int64_t cap = int64_t(sm_count) * 32;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        const bool narrow = s.total_keep < (int64_t(1) << 31);
#define BTC_ISO_VEC(LOG_L)                                                                                     \
        do {                                                                                                   \
            if (narrow) isolated_sum_vector_kernel<R, CPLX, LOG_L, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);   \
            else isolated_sum_vector_kernel<R, CPLX, LOG_L, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);           \
        } while (0)
        switch (log_l) {
        case 3: BTC_ISO_VEC(3); break;
        case 2: BTC_ISO_VEC(2); break;
        case 1: BTC_ISO_VEC(1); break;
        default: BTC_ISO_VEC(0); break;
        }
#undef BTC_ISO_VEC
        return cudaGetLastError();
    }
    const int lanes = s.lanes_over_iso ? 32 : 1;
    int64_t blocks = (s.total_keep * lanes + 255) / 256;
    const int64_t cap = int64_t(sm_count) * 32;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    const bool narrow = s.total_keep < (int64_t(1) << 31) && s.total_iso < (int64_t(1) << 31);   // indices fit 32 bits
    if (lanes == 32) {
        if (narrow) isolated_sum_kernel<R, CPLX, 32, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);
        else isolated_sum_kernel<R, CPLX, 32, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);
    } else {
        if (narrow) isolated_sum_kernel<R, CPLX, 1, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);
        else isolated_sum_kernel<R, CPLX, 1, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t run_isolated_sum(btc_dtype_t dt, const IsolatedSum &s, const void *src, void *dst, int sm_count, cudaStream_t st)
{
    switch (dt) {
    case BTC_F32: return launch_isolated_sum<float, false>(s, src, dst, sm_count, st);
    case BTC_F64: return launch_isolated_sum<double, false>(s, src, dst, sm_count, st);
    case BTC_C32: return launch_isolated_sum<float, true>(s, src, dst, sm_count, st);
    default: return launch_isolated_sum<double, true>(s, src, dst, sm_count, st);
    }
}

bool is_zero(const double v[2]) { return v[0] == 0.0 && v[1] == 0.0; }

template <typename R, bool CPLX>
cudaError_t launch_generic(const GenericParams &gp, int blocks, bool warp_per_elem, cudaStream_t st)
{
    if (warp_per_elem) generic_contract_kernel<R, CPLX, 32><<<blocks, 256, 0, st>>>(gp);
    else generic_contract_kernel<R, CPLX, 1><<<blocks, 256, 0, st>>>(gp);
    return cudaGetLastError();
}

}  // namespace

// =================================================================================== C ABI
extern "C" {

btc_error_t btc_create_handle(btc_handle_t *out)
{
    if (!out) return BTC_ERR_INVALID_ARGUMENT;
    btc_handle_s *h = new (std::nothrow) btc_handle_s;
    if (!h) return BTC_ERR_OUT_OF_MEMORY;
    int dev = -1;
    if (cudaGetDevice(&dev) == cudaSuccess && dev >= 0) {
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0) {
            h->device = dev;
            h->sm_count = sms;
        }
    }
    cudaGetLastError();   // a machine without a GPU still gets a handle that can validate and plan
    *out = h;
    return BTC_SUCCESS;
}

btc_error_t btc_destroy_handle(btc_handle_t *handle)
{
    if (!handle) return BTC_ERR_INVALID_ARGUMENT;
    delete *handle;
    *handle = nullptr;
    return BTC_SUCCESS;
}

btc_error_t btc_create_tensor_info(btc_handle_t handle, btc_dtype_t dtype, int32_t rank, const int64_t *extents,
                                   const int64_t *strides, btc_tensor_info_t *out)
{
    if (!handle || !out) return BTC_ERR_INVALID_ARGUMENT;
    if (rank < 0 || rank > BTC_MAX_RANK) return BTC_ERR_INVALID_ARGUMENT;
    if (int(dtype) < 0 || int(dtype) > int(BTC_C64)) return BTC_ERR_INVALID_ARGUMENT;
    if (rank > 0 && !extents) return BTC_ERR_INVALID_ARGUMENT;
    for (int i = 0; i < rank; ++i)
        if (extents[i] < 1) return BTC_ERR_INVALID_EXTENT;
    btc_tensor_info_s *t = new (std::nothrow) btc_tensor_info_s;
    if (!t) return BTC_ERR_OUT_OF_MEMORY;
    t->desc.dtype = dtype;
    t->desc.extent.assign(extents, extents + rank);
    if (strides) {
        t->desc.stride.assign(strides, strides + rank);
    } else {
        int64_t s = 1;
        for (int i = 0; i < rank; ++i) {
            t->desc.stride.push_back(s);
            s *= extents[i];
        }
    }
    *out = t;
    return BTC_SUCCESS;
}

btc_error_t btc_destroy_tensor_info(btc_tensor_info_t *info)
{
    if (!info) return BTC_ERR_INVALID_ARGUMENT;
    delete *info;
    *info = nullptr;
    return BTC_SUCCESS;
}

btc_error_t btc_create_contraction(btc_handle_t handle, btc_tensor_info_t A, const int64_t *labelsA, int conjA,
                                   btc_tensor_info_t B, const int64_t *labelsB, int conjB, btc_tensor_info_t C,
                                   const int64_t *labelsC, int conjC, btc_tensor_info_t D, const int64_t *labelsD,
                                   const void *alpha, const void *beta, btc_contraction_t *out)
{
    if (!handle || !A || !B || !D || !out) return BTC_ERR_INVALID_ARGUMENT;
    if ((!labelsA && !A->desc.extent.empty()) || (!labelsB && !B->desc.extent.empty()) ||
        (!labelsD && !D->desc.extent.empty()) || (C && !labelsC && !C->desc.extent.empty()))
        return BTC_ERR_INVALID_ARGUMENT;
    btc_contraction_s *op = new (std::nothrow) btc_contraction_s;
    if (!op) return BTC_ERR_OUT_OF_MEMORY;
    op->handle = *handle;
    op->req.A = A->desc;
    op->req.B = B->desc;
    op->req.D = D->desc;
    op->req.labelsA.assign(labelsA, labelsA + A->desc.extent.size());
    op->req.labelsB.assign(labelsB, labelsB + B->desc.extent.size());
    op->req.labelsD.assign(labelsD, labelsD + D->desc.extent.size());
    op->req.has_c = C != nullptr;
    if (C) {
        op->req.C = C->desc;
        op->req.labelsC.assign(labelsC, labelsC + C->desc.extent.size());
    }
    op->req.conjA = conjA != 0;
    op->req.conjB = conjB != 0;
    op->req.conjC = conjC != 0;
    if (alpha) to_double2(D->desc.dtype, alpha, op->alpha);
    if (beta) to_double2(D->desc.dtype, beta, op->beta);
    if (!C && !is_zero(op->beta)) {
        delete op;
        return BTC_ERR_INVALID_ARGUMENT;
    }
    const int rc = replan(op);
    if (rc != BTC_SUCCESS) {
        free_tables(op);
        delete op;
        return rc;
    }
    if (std::getenv("BTC_LOG")) {
        std::fprintf(stderr, "[btc] %s\n", op->plan.describe().c_str());
        // a large problem on the per-element kernel is almost always an unintended fall-back: say so
        const Plan &pl = op->plan;
        const double flops = 2.0 * double(pl.Bt) * double(pl.M) * double(pl.N) * double(pl.K);
        if (pl.kernel == BTC_KERNEL_GENERIC && flops > 1e9)
            std::fprintf(stderr, "[btc] note: %.3g flop on the per-element kernel (no tiled plan fits: offset tables too large, "
                                 "mixed element types, or forced by attribute)\n", flops);
    }
    *out = op;
    return BTC_SUCCESS;
}

btc_error_t btc_destroy_contraction(btc_contraction_t *op)
{
    if (!op) return BTC_ERR_INVALID_ARGUMENT;
    if (*op) {
        free_host_pipeline(*op);
        free_real_form(*op);
        free_tables(*op);
        delete *op;
    }
    *op = nullptr;
    return BTC_SUCCESS;
}

btc_error_t btc_contraction_workspace_size(btc_contraction_t op, size_t *bytes)
{
    if (!op || !bytes) return BTC_ERR_INVALID_ARGUMENT;
    *bytes = op->workspace_bytes;
    return BTC_SUCCESS;
}

btc_error_t btc_set_attr(btc_contraction_t op, int32_t key, const void *value, size_t len)
{
    if (!op || !value) return BTC_ERR_INVALID_ARGUMENT;
    if (len != sizeof(int32_t)) return BTC_ERR_INVALID_ARGUMENT;
    int32_t v;
    std::memcpy(&v, value, sizeof v);
    if (key == BTC_ATTR_POLL_LIMIT) {            // no re-planning: the next execute uses it
        if (v < 0) return BTC_ERR_INVALID_ARGUMENT;
        op->poll_limit = uint32_t(v);
        return BTC_SUCCESS;
    }
    if (key == BTC_ATTR_DEVICE_ERROR) {          // writing 0 clears the device error word
        if (v != 0) return BTC_ERR_INVALID_ARGUMENT;
        if ((op->d_error && cudaMemset(op->d_error, 0, sizeof(int32_t)) != cudaSuccess) ||
            (op->real_inner && op->real_inner->d_error && cudaMemset(op->real_inner->d_error, 0, sizeof(int32_t)) != cudaSuccess)) {
            cudaGetLastError();
            return BTC_ERR_CUDA;
        }
        return BTC_SUCCESS;
    }
    const PlanRequest saved = op->req;
    const bool saved_pre_reduce = op->pre_reduce;
    if (key == BTC_ATTR_PRE_REDUCE) {
        if (v != 0 && v != 1) return BTC_ERR_INVALID_ARGUMENT;
        op->pre_reduce = v != 0;
    } else if (key == BTC_ATTR_KERNEL) {
        if (v < BTC_KERNEL_AUTO || v > BTC_KERNEL_TILED) return BTC_ERR_INVALID_ARGUMENT;
        op->req.force_kernel = v;
    } else if (key == BTC_ATTR_VARIANT) {
        op->req.force_variant = v;
    } else if (key == BTC_ATTR_SPLIT_K) {
        if (v < 0) return BTC_ERR_INVALID_ARGUMENT;
        op->req.force_split_k = v;
    } else if (key == BTC_ATTR_COMPUTE_PRECISION) {
        if (v != BTC_PRECISION_DEFAULT && v != BTC_PRECISION_STRICT && v != BTC_PRECISION_FP64_SUMS) return BTC_ERR_INVALID_ARGUMENT;
        if (v == BTC_PRECISION_STRICT && op->plan.dtype == BTC_C32) return BTC_ERR_NOT_SUPPORTED;
        op->req.strict_fp32 = v;
    } else if (key == BTC_ATTR_BATCH_HINT) {
        if (v < 1) return BTC_ERR_INVALID_ARGUMENT;
        op->req.batch_hint = v;
    } else {
        return BTC_ERR_INVALID_ARGUMENT;
    }
    free_host_pipeline(op);    // built for the previous plan
    int rc = replan(op);
    if (rc != BTC_SUCCESS) {   // keep the object usable with its previous plan
        op->req = saved;
        op->pre_reduce = saved_pre_reduce;
        replan(op);
    }
    return rc;
}

btc_error_t btc_get_attr(btc_contraction_t op, int32_t key, void *value, size_t len, size_t *needed)
{
    if (!op) return BTC_ERR_INVALID_ARGUMENT;
    int32_t i32[4];
    int64_t i64[4];
    const void *src = i32;
    size_t n = 0;
    const Plan &pl = op->plan;
    // what runs: for complex64 operations in their real form, the fp32 operation's kernel, tile, grid
    const btc_contraction_s *run = op->real_inner ? op->real_inner : op;
    const Plan &rp = run->plan;
    switch (key) {
    case BTC_ATTR_KERNEL: i32[0] = rp.kernel; n = 4; break;
    case BTC_ATTR_SPLIT_K: i32[0] = rp.split_k; n = 4; break;
    case BTC_ATTR_TILE: i32[0] = rp.tile.bm; i32[1] = rp.tile.bn; i32[2] = rp.tile.bk; n = 12; break;
    case BTC_ATTR_GROUPS: i64[0] = pl.Bt; i64[1] = pl.M; i64[2] = pl.N; i64[3] = pl.K; src = i64; n = 32; break;
    case BTC_ATTR_GRID: i32[0] = run->grid[0]; i32[1] = run->grid[1]; i32[2] = run->grid[2]; n = 12; break;
    case BTC_ATTR_NUM_MODES:
        i32[0] = int32_t(pl.batch.size()); i32[1] = int32_t(pl.m.size());
        i32[2] = int32_t(pl.n.size()); i32[3] = int32_t(pl.k.size()); n = 16; break;
    case BTC_ATTR_SWAPPED: i32[0] = pl.swapped ? 1 : 0; n = 4; break;
    case BTC_ATTR_VARIANT: i32[0] = rp.tile.variant; n = 4; break;
    case BTC_ATTR_PRE_REDUCE: i32[0] = (op->sumA.active ? 1 : 0) | (op->sumB.active ? 2 : 0); n = 4; break;
    case BTC_ATTR_BATCH_HINT: i32[0] = op->req.batch_hint; n = 4; break;
    case BTC_ATTR_COMPUTE_PRECISION: i32[0] = op->req.strict_fp32; n = 4; break;
    case BTC_ATTR_DEVICE_ERROR:
        i32[0] = 0;
        for (const btc_contraction_s *o : {static_cast<const btc_contraction_s *>(op), static_cast<const btc_contraction_s *>(op->real_inner)}) {
            if (!o || !o->d_error || i32[0] != 0) continue;
            if (cudaMemcpy(&i32[0], o->d_error, sizeof(int32_t), cudaMemcpyDeviceToHost) != cudaSuccess) {
                cudaGetLastError();
                return BTC_ERR_CUDA;
            }
        }
        n = 4;
        break;
    default: return BTC_ERR_INVALID_ARGUMENT;
    }
    if (needed) *needed = n;
    if (!value) return needed ? BTC_SUCCESS : BTC_ERR_INVALID_ARGUMENT;
    if (len < n) return BTC_ERR_INVALID_ARGUMENT;
    std::memcpy(value, src, n);
    return BTC_SUCCESS;
}

namespace {
// Pointer-array batch seen by the tiled kernels: `count` times the operation's own batch entries,
// with offset tables (elements, relative to entry 0's pointers) that live in the caller's workspace.
struct BatchView {
    int64_t count;
    const int64_t *offA_h, *offB_h, *offD_h;   // [count * Bt], planned roles
    const int64_t *host_tab = nullptr;         // the same three tables on the host, when they ride in the kernel's parameters instead
    void *partials;
    bool aligned16_D, aligned_A, aligned_B;     // every entry's pointer keeps the vector alignment
    bool aligned16_A;                           // every entry's M-side input pointer is 16-byte aligned
};

btc_error_t execute_impl(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *A, const void *B,
                         const void *beta, const void *C, void *D, void *workspace, size_t workspace_bytes,
                         btc_status_t *status, const BatchView *bv);
}  // namespace

btc_error_t btc_execute(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *A, const void *B,
                        const void *beta, const void *C, void *D, void *workspace, size_t workspace_bytes,
                        btc_status_t *status)
{
    return execute_impl(op, cuda_stream, alpha, A, B, beta, C, D, workspace, workspace_bytes, status, nullptr);
}

namespace {
// Spans of the tensors the kernels address, in planned roles (a Case 4 input that was summed first is
// the dense result of that sum); a pointer-array batch reaches other buffers, so its spans are left open.
void fill_spans(const btc_contraction_s *op, OffsetSpans &sp, bool open = false)
{
    const int64_t big = int64_t(1) << 62;
    int64_t lo[2] = {op->spanA_lo, op->spanB_lo}, hi[2] = {op->spanA_hi, op->spanB_hi};
    if (op->sumA.active) { lo[0] = 0; hi[0] = op->sumA.total_keep - 1; }
    if (op->sumB.active) { lo[1] = 0; hi[1] = op->sumB.total_keep - 1; }
    const int a = op->plan.swapped ? 1 : 0;
    sp.lo[0] = lo[a]; sp.hi[0] = hi[a]; sp.lo[1] = lo[1 - a]; sp.hi[1] = hi[1 - a];
    sp.lo[2] = op->spanD_lo; sp.hi[2] = op->spanD_hi;
    if (open)
        for (int i = 0; i < 3; ++i) { sp.lo[i] = -big; sp.hi[i] = big; }
    sp.error_word = op->d_error;
}

btc_error_t execute_impl(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *A, const void *B,
                         const void *beta, const void *C, void *D, void *workspace, size_t workspace_bytes,
                         btc_status_t *status, const BatchView *bv)
{
    if (!op || !D) return BTC_ERR_INVALID_ARGUMENT;
    if (op->handle.device < 0) return BTC_ERR_CUDA;   // no device: nothing can run, and nothing else will
    const Plan &pl = op->plan;
    double al[2] = {op->alpha[0], op->alpha[1]}, be[2] = {op->beta[0], op->beta[1]};
    if (alpha) to_double2(pl.dtype, alpha, al);
    if (beta) to_double2(pl.dtype, beta, be);
    const bool use_ab = !is_zero(al), use_c = !is_zero(be);
    if (use_ab && (!A || !B)) return BTC_ERR_INVALID_ARGUMENT;
    if (use_c && (!C || !pl.has_c_desc)) return BTC_ERR_INVALID_ARGUMENT;
    auto misaligned = [&](const void *p, size_t a) { return p && (reinterpret_cast<uintptr_t>(p) % a) != 0; };
    // complex128 accesses are 16-byte wide; everything else needs its element alignment
    auto need_of = [](btc_dtype_t t) -> size_t { return t == BTC_C64 ? 16 : (t == BTC_C32 ? 8 : dtype_size(t)); };
    const size_t need = need_of(pl.dtype);
    if (misaligned(A, need_of(op->req.A.dtype)) || misaligned(B, need_of(op->req.B.dtype)) ||
        misaligned(C, need_of(op->req.has_c ? op->req.C.dtype : pl.dtype)) || misaligned(D, need))
        return BTC_ERR_MISALIGNED;
    if (op->workspace_floor > 0 && !bv) {        // a pointer-array batch has checked its own layout
        if (!workspace || workspace_bytes < op->workspace_floor) return BTC_ERR_WORKSPACE_TOO_SMALL;
        if (misaligned(workspace, 256)) return BTC_ERR_MISALIGNED;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // complex64 through its real form on the fp32 tensor-core kernels: expand the smaller input (alpha and
    // both conjugations go into it), then run the real contraction over the float views of the other
    // tensors.  Needs a real beta and C as it is; pointer-array calls keep the complex kernels.
    if (op->real_inner && op->real_view_only) {
        // mixed element types through the real views (build_mixed_real_view): real scalars, C as it is,
        // and room for the real operation's own scratch; otherwise the per-element kernel below
        btc_contraction_s *in = op->real_inner;
        const bool room = in->workspace_floor == 0 || (workspace && !misaligned(workspace, 256) && workspace_bytes >= in->workspace_floor);
        if (!bv && al[1] == 0.0 && be[1] == 0.0 && !(use_c && op->req.conjC) && room) {
            in->poll_limit = op->poll_limit;
            const float af = float(al[0]), bf = float(be[0]);
            const bool f32 = in->plan.dtype == BTC_F32;
            return execute_impl(in, cuda_stream, f32 ? static_cast<const void *>(&af) : static_cast<const void *>(&al[0]), A, B,
                                f32 ? static_cast<const void *>(&bf) : static_cast<const void *>(&be[0]), use_c ? C : nullptr, D,
                                workspace, workspace_bytes, status, nullptr);
        }
    } else if (op->real_inner && !bv && use_ab && be[1] == 0.0 && !(use_c && pl.conjC) && workspace && !misaligned(workspace, 256) &&
        workspace_bytes >= op->real_x_bytes + op->real_inner->workspace_bytes) {
        ComplexExpandParams ep = op->real_expand;
        ep.src = static_cast<const float2 *>(op->real_expand_A ? A : B);
        ep.dst = static_cast<float *>(workspace);
        ep.alpha_r = float(al[0]); ep.alpha_i = float(al[1]);
        ep.conj_x = (op->real_expand_A ? op->req.conjA : op->req.conjB) ? 1 : 0;
        ep.conj_y = (op->real_expand_A ? op->req.conjB : op->req.conjA) ? 1 : 0;
        int64_t blocks = (ep.total + 255) / 256;
        const int64_t cap = int64_t(op->handle.sm_count) * 16;
        if (blocks > cap) blocks = cap;
        complex_expand_kernel<<<unsigned(blocks), 256, 0, st>>>(ep);
        if (cudaGetLastError() != cudaSuccess) return BTC_ERR_CUDA;
        const float one = 1.f, beta_r = float(be[0]);
        const void *pa = op->real_expand_A ? workspace : A, *pb = op->real_expand_A ? B : workspace;
        btc_contraction_s *in = op->real_inner;
        in->poll_limit = op->poll_limit;
        const btc_error_t rc = execute_impl(in, cuda_stream, &one, pa, pb, &beta_r, use_c ? C : nullptr, D,
                                            static_cast<char *>(workspace) + op->real_x_bytes, workspace_bytes - op->real_x_bytes,
                                            status, nullptr);
        if (rc == BTC_SUCCESS && status && *status) (*status)->launches += 1;
        return rc;
    }
    int launches = 0;
    int ran_variant = op->plan.kernel == BTC_KERNEL_TILED ? op->plan.tile.variant : -1;
    cudaError_t ce = cudaSuccess;
    // Case 4: sum the inputs over their isolated labels first; the contraction then reads A', B'
    if (use_ab && op->sumA.active) {
        ce = run_isolated_sum(pl.dtype, op->sumA, A, workspace, op->handle.sm_count, st);
        if (ce != cudaSuccess) return BTC_ERR_CUDA;
        A = workspace;
        ++launches;
    }
    if (use_ab && op->sumB.active) {
        void *dst = static_cast<char *>(workspace) + op->sumB_offset;
        ce = run_isolated_sum(pl.dtype, op->sumB, B, dst, op->handle.sm_count, st);
        if (ce != cudaSuccess) return BTC_ERR_CUDA;
        B = dst;
        ++launches;
    }
    const void *pA = pl.swapped ? B : A, *pB = pl.swapped ? A : B;

    if (pl.kernel == BTC_KERNEL_GENERIC || !use_ab) {
        GenericParams gp;
        std::memset(&gp, 0, sizeof gp);
        gp.A = pA; gp.B = pB; gp.C = C; gp.D = D;
        int nd = 0;
        for (auto *g : {&pl.batch, &pl.m, &pl.n})
            for (auto &md : *g) {
                gp.ext_d[nd] = md.extent; gp.sA_d[nd] = md.sA; gp.sB_d[nd] = md.sB; gp.sD_d[nd] = md.sD;
                ++nd;
            }
        if (nd > kGenericMaxD || pl.k.size() > size_t(kGenericMaxK)) return BTC_ERR_NOT_SUPPORTED;
        gp.nd = nd;
        gp.nk = int32_t(pl.k.size());
        for (int i = 0; i < gp.nk; ++i) {
            gp.ext_k[i] = pl.k[size_t(i)].extent; gp.sA_k[i] = pl.k[size_t(i)].sA; gp.sB_k[i] = pl.k[size_t(i)].sB;
        }
        gp.total_d = pl.Bt * pl.M * pl.N;
        gp.total_k = pl.K;
        gp.alpha[0] = al[0]; gp.alpha[1] = al[1]; gp.beta[0] = be[0]; gp.beta[1] = be[1];
        gp.conjA = pl.conjA; gp.conjB = pl.conjB; gp.conjC = pl.conjC;
        gp.cplxA = pl.cplxA; gp.cplxB = pl.cplxB; gp.cplxC = pl.cplxC;
        gp.use_ab = use_ab; gp.use_c = use_c;
        fill_spans(op, gp.spans);
        bool wpe = pl.kernel == BTC_KERNEL_GENERIC && op->grid[1] == 32;
        int blocks = op->grid[0];
        if (pl.kernel != BTC_KERNEL_GENERIC) {   // alpha == 0 on a tiled plan: D = beta * op(C)
            int64_t b = (gp.total_d + 255) / 256, cap = int64_t(op->handle.sm_count) * 32;
            blocks = int(b < cap ? (b < 1 ? 1 : b) : cap);
        }
        switch (pl.dtype) {
        case BTC_F32: ce = launch_generic<float, false>(gp, blocks, wpe, st); break;
        case BTC_F64: ce = launch_generic<double, false>(gp, blocks, wpe, st); break;
        case BTC_C32: ce = launch_generic<float, true>(gp, blocks, wpe, st); break;
        case BTC_C64: ce = launch_generic<double, true>(gp, blocks, wpe, st); break;
        }
        launches += 1;
    } else {
        TiledParams tp;
        std::memset(&tp, 0, sizeof tp);
        tp.A = pA; tp.B = pB; tp.C = C; tp.D = D;
        tp.offA_m = op->d_offA_m; tp.offD_m = op->d_offD_m; tp.offB_n = op->d_offB_n; tp.offD_n = op->d_offD_n;
        tp.offA_k = op->d_offA_k; tp.offB_k = op->d_offB_k;
        tp.offA_h = op->d_offA_h; tp.offB_h = op->d_offB_h; tp.offD_h = op->d_offD_h;
        tp.M = pl.M; tp.N = pl.N; tp.K = pl.K; tp.Bt = pl.Bt;
        tp.tiles_m = op->tiles_m; tp.tiles_n = op->tiles_n; tp.raster_n_fast = op->raster_n_fast;
        tp.bm = pl.tile.bm; tp.bn = pl.tile.bn;
        tp.split_k = pl.split_k; tp.k_per_split = op->k_per_split;
        tp.dirA = int32_t(pl.dirA); tp.dirB = int32_t(pl.dirB);
        // vector copies need the base pointers aligned as well
        tp.vecA = (misaligned(pA, size_t(pl.alignA)) || (bv && !bv->aligned_A)) ? 1 : pl.vecA;
        tp.vecB = (misaligned(pB, size_t(pl.alignB)) || (bv && !bv->aligned_B)) ? 1 : pl.vecB;
        tp.conjA = pl.conjA; tp.conjB = pl.conjB; tp.conjC = pl.conjC;
        tp.use_c = use_c;
        tp.alpha[0] = al[0]; tp.alpha[1] = al[1]; tp.beta[0] = be[0]; tp.beta[1] = be[1];
        tp.partials = workspace ? static_cast<char *>(workspace) + op->partials_offset : nullptr;
        tp.error_word = op->d_error;
        tp.poll_limit = op->poll_limit;
        fill_spans(op, tp.spans, bv != nullptr);
        tp.tmaA_coord_m = op->d_tma_coord_m; tp.tmaA_coord_k = op->d_tma_coord_k; tp.tmaA_coord_h = op->d_tma_coord_h;
        tp.skinny_orderA = op->d_skinny_order[0]; tp.skinny_orderB = op->d_skinny_order[3];
        tp.skinny_regular = op->skinny_regular ? 1 : 0;
        int64_t ctas = op->grid[0];
        int64_t reduce_ctas = (ctas / pl.split_k) * ((int64_t(pl.tile.bm) * pl.tile.bn + 1023) / 1024);
        // 16-byte stores of D (and loads of C) need those base pointers aligned too
        tp.vecD = (pl.vecD == 4 && !misaligned(D, 16) && !(use_c && misaligned(C, 16)) && !(bv && !bv->aligned16_D)) ? 4 : 1;
        const bool persistent = pl.dtype == BTC_F32 && f32_persistent(pl.tile.variant);
        if (bv) {
            // the pointer array multiplies the batch entries; everything else of the plan stands
            tp.Bt = pl.Bt * bv->count;
            tp.offA_h = bv->offA_h; tp.offB_h = bv->offB_h; tp.offD_h = bv->offD_h;
            tp.partials = bv->partials;
            const int64_t work = int64_t(op->tiles_m) * op->tiles_n * pl.split_k * tp.Bt;
            if (work > 0x7fffffffLL) return BTC_ERR_NOT_SUPPORTED;
            ctas = persistent ? (work < op->handle.sm_count ? work : op->handle.sm_count) : work;
            reduce_ctas = (work / pl.split_k) * ((int64_t(pl.tile.bm) * pl.tile.bn + 1023) / 1024);
        }
        // fp64 kernels, launches of at most one wave (the latency-bound small problems): 2, 4 or 8 k slices of a
        // tile run as one thread-block cluster, one launch and no scratch.  Larger grids keep the two-kernel
        // form: clusters of CTAs that each fill an SM schedule worse there (workload 6: 1.44 ms against 1.30 ms).
        tp.cluster_split = ((pl.dtype == BTC_F64 || pl.dtype == BTC_C64) && (pl.split_k == 2 || pl.split_k == 4 || pl.split_k == 8) &&
                            ctas <= op->handle.sm_count) ? 1 : 0;
        if (pl.tile.variant == kStreamVariant) {
            // 16-byte accesses along the first M mode where the plan's strides and these pointers allow
            const bool vec_d = pl.rows16D && !misaligned(D, 16) && !(use_c && misaligned(C, 16)) && !(bv && !bv->aligned16_D);
            const bool vec_a = vec_d && pl.rows16A && !misaligned(pA, 16) && !(bv && !bv->aligned16_A);
            ce = launch_stream(tp, int(pl.dtype), vec_d, vec_a, op->handle.sm_count, st);
        } else if (pl.dtype == BTC_F32) {
            switch (pl.tile.variant) {
            case 0: ce = launch_tiled_f32<F32Big>(tp, ctas, reduce_ctas, st); break;
            case 1: ce = launch_tiled_f32<F32Small>(tp, ctas, reduce_ctas, st); break;
            case 2: ce = launch_tiled_f32<F32Wide>(tp, ctas, reduce_ctas, st); break;
            case 3: ce = launch_tiled_f32<F32BigP>(tp, ctas, reduce_ctas, st); break;
            case 4: ce = launch_tiled_f32<F32WideP>(tp, ctas, reduce_ctas, st); break;
            case 5: ce = launch_tiled_f32<F32Big32>(tp, ctas, reduce_ctas, st); break;
            case 6: ce = launch_tiled_tf32<F32Tc>(tp, ctas, reduce_ctas, st); break;
            case 7: ce = launch_tiled_tf32<F32TcSmall>(tp, ctas, reduce_ctas, st); break;
            case 22: ce = launch_tiled_tf32<F32TcTiny>(tp, ctas, reduce_ctas, st); break;
            case 23:
                // 16-byte pieces need 16-byte aligned operands; otherwise the mma.sync kernel with the same tiles
                if (tp.vecA != 4 || tp.vecB != 4) {
                    ran_variant = 6;
                    ce = launch_tiled_tf32<F32Tc>(tp, int64_t(op->tiles_m) * op->tiles_n * tp.Bt, reduce_ctas, st);
                } else {
                    // Where D's contiguous runs along m are short (interleaved small modes) the kernel runs
                    // with the roles exchanged: D's smallest-stride label on its column side, so that each
                    // thread writes 16-byte pieces and neighbouring threads neighbouring pieces.  With long
                    // runs a warp's 32 consecutive rows of one column are a whole line as they are.
                    TiledParams sp = tp;
                    SkinnyBatch sb;
                    sb.count = 0; sb.pad = 0;
                    const int64_t *tabA = nullptr, *tabB = nullptr;
                    if (bv && bv->host_tab) {
                        sb.count = int32_t(tp.Bt);
                        tabA = bv->host_tab; tabB = bv->host_tab + tp.Bt;
                        std::memcpy(sb.offD_h, bv->host_tab + 2 * tp.Bt, size_t(tp.Bt) * sizeof(int64_t));
                    }
                    if (tp.vecD == 4 && op->skinny_run_m < 32) {
                        std::swap(tabA, tabB);
                        std::swap(sp.A, sp.B);
                        std::swap(sp.offA_m, sp.offB_n); std::swap(sp.offD_m, sp.offD_n);
                        std::swap(sp.offA_k, sp.offB_k); std::swap(sp.offA_h, sp.offB_h);
                        std::swap(sp.M, sp.N); std::swap(sp.tiles_m, sp.tiles_n);
                        std::swap(sp.dirA, sp.dirB); std::swap(sp.vecA, sp.vecB);
                        std::swap(sp.conjA, sp.conjB);
                        std::swap(sp.spans.lo[0], sp.spans.lo[1]); std::swap(sp.spans.hi[0], sp.spans.hi[1]);
                        sp.skinny_orderA = op->d_skinny_order[2]; sp.skinny_orderB = op->d_skinny_order[1];
                        sp.skinny_vec_n = 4;
                    }
                    // D's column offsets inside a tile, when every tile's columns are laid out alike
                    const bool exchanged = sp.skinny_vec_n == 4;
                    const std::vector<int64_t> &col_off = exchanged ? pl.offD_m : pl.offD_n;
                    sp.skinny_d_regular = op->skinny_d_regular[exchanged ? 0 : 1] ? 1 : 0;
                    for (size_t c = 0; c < 128; ++c) sp.skinny_col_rel[c] = c < col_off.size() ? int32_t(col_off[c] - col_off[0]) : 0;
                    if (sb.count) {
                        std::memcpy(sb.offA_h, tabA, size_t(tp.Bt) * sizeof(int64_t));
                        std::memcpy(sb.offB_h, tabB, size_t(tp.Bt) * sizeof(int64_t));
                    }
                    ce = launch_skinny_umma(sp, sb, int(ctas), st);
                }
                break;
            case 8: ce = launch_tiled_tf32<F32TcWide>(tp, ctas, reduce_ctas, st); break;
            case 9: ce = launch_tiled_tf32<F32TcMid>(tp, ctas, reduce_ctas, st); break;
            case 10: ce = launch_umma<F32Umma96>(tp, ctas, st); break;
            case 11: ce = launch_umma<F32Umma128>(tp, ctas, st); break;
            case 12: ce = launch_umma<F32Umma256>(tp, ctas, st); break;
            case 13: ce = launch_umma<F32Umma96T>(tp, ctas, st); break;
            case 14: ce = launch_umma<F32Umma128T>(tp, ctas, st); break;
            case 15: ce = launch_umma<F32Umma96T2>(tp, ctas, st); break;
            case 16: ce = launch_umma<F32Umma128T2>(tp, ctas, st); break;
            default: {
                // bulk tensor copies need a 16-byte aligned base and a description the driver accepts;
                // otherwise the gathering variant with the same tile runs
                CUtensorMap mapA;
                const int v = pl.tile.variant;
                if (bv || misaligned(pA, 16) || !encode_tma_operand(op->tmaA, pA, &mapA)) {   // (a pointer array is no box dimension)
                    ran_variant = (v <= 18 || v == 21) ? 13 : 14;
                    ce = ran_variant == 13 ? launch_umma<F32Umma96T>(tp, ctas, st) : launch_umma<F32Umma128T>(tp, ctas, st);
                }
                else if (v == 17) ce = launch_umma<F32Umma96B24>(tp, ctas, st, &mapA);
                else if (v == 18) ce = launch_umma<F32Umma96B32>(tp, ctas, st, &mapA);
                else if (v == 19) ce = launch_umma<F32Umma128B32>(tp, ctas, st, &mapA);
                else if (v == 21) ce = launch_umma<F32Umma96B24x2>(tp, ctas, st, &mapA);
                else ce = launch_umma<F32Umma128B24>(tp, ctas, st, &mapA);
            } break;
            }
        } else if (pl.dtype == BTC_C32) {
            ce = pl.tile.variant == 0 ? launch_tiled_tf32<C32Tc>(tp, ctas, reduce_ctas, st)
                                      : launch_tiled_tf32<C32TcSmall>(tp, ctas, reduce_ctas, st);
        } else if (pl.dtype == BTC_F64)
            switch (pl.tile.variant) {
            case 0: ce = launch_tiled<F64Big>(tp, ctas, reduce_ctas, st); break;
            case 1: ce = launch_tiled<F64Small>(tp, ctas, reduce_ctas, st); break;
            case 2: ce = launch_tiled<F64Big16>(tp, ctas, reduce_ctas, st); break;
            case 3: ce = launch_tiled<F64Big3>(tp, ctas, reduce_ctas, st); break;
            default: ce = launch_tiled<F64BigT>(tp, ctas, reduce_ctas, st); break;
            }
        else
            ce = pl.tile.variant == 0 ? launch_tiled<C64Big>(tp, ctas, reduce_ctas, st)
                 : (pl.tile.variant == 1 ? launch_tiled<C64Small>(tp, ctas, reduce_ctas, st)
                                         : launch_tiled<C64Big16>(tp, ctas, reduce_ctas, st));
        launches += (pl.split_k > 1 && !tp.cluster_split) ? 2 : 1;
    }
    if (ce != cudaSuccess) return BTC_ERR_CUDA;
    if (status) {
        btc_status_s *s = new (std::nothrow) btc_status_s;
        if (!s) return BTC_ERR_OUT_OF_MEMORY;
        s->kernel = use_ab ? pl.kernel : BTC_KERNEL_GENERIC;
        s->launches = launches;
        s->variant = ran_variant;
        s->split_k = pl.split_k;
        s->grid[0] = op->grid[0]; s->grid[1] = op->grid[1]; s->grid[2] = op->grid[2];
        *status = s;
    }
    return BTC_SUCCESS;
}

// one launch serves the whole pointer array: tiled plan, both inputs read as they are
bool batch_in_one_launch(const btc_contraction_s *op)
{
    return op->plan.kernel == BTC_KERNEL_TILED && !op->sumA.active && !op->sumB.active;
}
size_t batch_tables_bytes(const btc_contraction_s *op, int64_t count)
{
    return (size_t(3) * size_t(count) * size_t(op->plan.Bt) * sizeof(int64_t) + 255) / 256 * 256;
}
}  // namespace

btc_error_t btc_contraction_batched_workspace_size(btc_contraction_t op, int64_t count, size_t *bytes)
{
    if (!op || !bytes || count < 1) return BTC_ERR_INVALID_ARGUMENT;
    if (!batch_in_one_launch(op)) { *bytes = op->workspace_bytes; return BTC_SUCCESS; }
    *bytes = batch_tables_bytes(op, count) + (op->workspace_floor - op->partials_offset) * size_t(count);
    return BTC_SUCCESS;
}

btc_error_t btc_execute_batched(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *const *A,
                                const void *const *B, const void *beta, const void *const *C, void *const *D,
                                int64_t count, void *workspace, size_t workspace_bytes)
{
    if (!op || !D || count < 1) return BTC_ERR_INVALID_ARGUMENT;
    if (op->handle.device < 0) return BTC_ERR_CUDA;
    const Plan &pl = op->plan;
    double al[2] = {op->alpha[0], op->alpha[1]}, be[2] = {op->beta[0], op->beta[1]};
    if (alpha) to_double2(pl.dtype, alpha, al);
    if (beta) to_double2(pl.dtype, beta, be);
    const bool use_ab = !is_zero(al), use_c = !is_zero(be);
    if ((use_ab && (!A || !B)) || (use_c && !C)) return BTC_ERR_INVALID_ARGUMENT;
    for (int64_t i = 0; i < count; ++i)
        if (!D[i] || (use_ab && (!A[i] || !B[i])) || (use_c && !C[i])) return BTC_ERR_INVALID_ARGUMENT;
    size_t need = 0;
    btc_contraction_batched_workspace_size(op, count, &need);
    if (need > 0 && (!workspace || workspace_bytes < need)) return BTC_ERR_WORKSPACE_TOO_SMALL;
    if (need > 0 && reinterpret_cast<uintptr_t>(workspace) % 256) return BTC_ERR_MISALIGNED;

    if (!batch_in_one_launch(op) || !use_ab) {
        // generic-kernel and Case 4 plans: one execute per entry, in order on the stream
        for (int64_t i = 0; i < count; ++i) {
            const btc_error_t rc = execute_impl(op, cuda_stream, alpha, use_ab ? A[i] : nullptr, use_ab ? B[i] : nullptr, beta,
                                                use_c ? C[i] : nullptr, D[i], workspace, workspace_bytes, nullptr, nullptr);
            if (rc != BTC_SUCCESS) return rc;
        }
        return BTC_SUCCESS;
    }

    // offsets of every entry relative to entry 0, in elements, added to the operation's own batch offsets
    const int64_t esz = int64_t(dtype_size(pl.dtype));
    const int64_t Bt = pl.Bt;
    std::vector<int64_t> tab(size_t(3) * size_t(count) * size_t(Bt));
    int64_t *tA = tab.data(), *tB = tA + count * Bt, *tD = tB + count * Bt;
    BatchView bv;
    bv.count = count;
    bv.aligned16_D = bv.aligned_A = bv.aligned_B = bv.aligned16_A = true;
    const void *const *pA = pl.swapped ? B : A, *const *pB = pl.swapped ? A : B;
    for (int64_t i = 0; i < count; ++i) {
        const int64_t dA = reinterpret_cast<intptr_t>(pA[i]) - reinterpret_cast<intptr_t>(pA[0]);
        const int64_t dB = reinterpret_cast<intptr_t>(pB[i]) - reinterpret_cast<intptr_t>(pB[0]);
        const int64_t dD = reinterpret_cast<intptr_t>(D[i]) - reinterpret_cast<intptr_t>(D[0]);
        if (dA % esz || dB % esz || dD % esz) return BTC_ERR_MISALIGNED;
        // C travels with D: one offset table serves both, so C[i] - C[0] must equal D[i] - D[0]
        if (use_c && reinterpret_cast<intptr_t>(C[i]) - reinterpret_cast<intptr_t>(C[0]) != dD) return BTC_ERR_NOT_SUPPORTED;
        bv.aligned_A = bv.aligned_A && reinterpret_cast<uintptr_t>(pA[i]) % size_t(pl.alignA) == 0;
        bv.aligned_B = bv.aligned_B && reinterpret_cast<uintptr_t>(pB[i]) % size_t(pl.alignB) == 0;
        bv.aligned16_A = bv.aligned16_A && reinterpret_cast<uintptr_t>(pA[i]) % 16 == 0;
        bv.aligned16_D = bv.aligned16_D && reinterpret_cast<uintptr_t>(D[i]) % 16 == 0 &&
                         (!use_c || reinterpret_cast<uintptr_t>(C[i]) % 16 == 0);
        for (int64_t h = 0; h < Bt; ++h) {
            tA[i * Bt + h] = pl.offA_h[size_t(h)] + dA / esz;
            tB[i * Bt + h] = pl.offB_h[size_t(h)] + dB / esz;
            tD[i * Bt + h] = pl.offD_h[size_t(h)] + dD / esz;
        }
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    // The short-K streaming kernel takes the offsets of up to 64 entries in its parameters: no copy before
    // the launch (which would also keep consecutive launches from overlapping their set-up).
    const bool in_params = pl.kernel == BTC_KERNEL_TILED && pl.dtype == BTC_F32 && pl.tile.variant == kSkinnyVariant &&
                           count * Bt <= kSkinnyInlineEntries && pl.vecA == 4 && pl.vecB == 4 && bv.aligned_A && bv.aligned_B;
    if (in_params) {
        bv.host_tab = tab.data();
    } else if (cudaMemcpyAsync(workspace, tab.data(), tab.size() * sizeof(int64_t), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return BTC_ERR_CUDA;
    }
    const int64_t *dtab = static_cast<const int64_t *>(workspace);
    bv.offA_h = dtab; bv.offB_h = dtab + count * Bt; bv.offD_h = dtab + 2 * count * Bt;
    bv.partials = static_cast<char *>(workspace) + batch_tables_bytes(op, count);
    return execute_impl(op, cuda_stream, alpha, A[0], B[0], beta, use_c ? C[0] : nullptr, D[0], workspace, workspace_bytes,
                        nullptr, &bv);
}

}  // extern "C"

namespace {

void free_host_pipeline(btc_contraction_s *op)
{
    HostPipeline *hp = op->host;
    if (!hp) return;
    for (int i = 0; i < 2; ++i) {
        if (hp->sub[i]) { free_tables(hp->sub[i]); delete hp->sub[i]; }
        if (hp->bufX[i]) cudaFree(hp->bufX[i]);
        if (hp->loaded[i]) cudaEventDestroy(hp->loaded[i]);
        if (hp->consumed[i]) cudaEventDestroy(hp->consumed[i]);
    }
    for (char *b : {hp->bufY, hp->bufD, hp->bufC, hp->ws}) if (b) cudaFree(b);
    if (hp->copy_stream) cudaStreamDestroy(hp->copy_stream);
    cudaGetLastError();
    delete hp;
    op->host = nullptr;
}

int position_of(const std::vector<int64_t> &labels, int64_t label)
{
    int at = -1;
    for (size_t i = 0; i < labels.size(); ++i)
        if (labels[i] == label) { if (at >= 0) return -2; at = int(i); }       // -2: repeated
    return at;
}

void span_of_desc(const TensorDesc &t, int64_t &lo, int64_t &hi)
{
    lo = hi = 0;
    for (size_t i = 0; i < t.extent.size(); ++i) {
        const int64_t d = t.stride[i] * (t.extent[i] - 1);
        if (d < 0) lo += d; else hi += d;
    }
}

// Decide how to cut the operation for host-buffer execution and build what that needs.  Not usable (the
// plain path runs) when no label qualifies or the slabs would overlap too much in memory.
void build_host_pipeline(btc_contraction_s *op)
{
    HostPipeline *hp = new (std::nothrow) HostPipeline;
    op->host = hp;
    if (!hp) return;
    hp->tried = true;
    const PlanRequest &rq = op->req;
    const size_t esz = dtype_size(rq.D.dtype);
    const int64_t spanA = op->spanA_hi - op->spanA_lo + 1, spanB = op->spanB_hi - op->spanB_lo + 1;
    hp->slab_is_A = spanA >= spanB;
    const TensorDesc &X = hp->slab_is_A ? rq.A : rq.B, &Y = hp->slab_is_A ? rq.B : rq.A;
    const std::vector<int64_t> &lX = hp->slab_is_A ? rq.labelsA : rq.labelsB, &lY = hp->slab_is_A ? rq.labelsB : rq.labelsA;
    if (size_t(std::max(spanA, spanB)) * esz < (size_t(64) << 20)) return;       // small inputs: one copy is as good
    // the label with the largest stride in the cut input that occurs once there and at most once elsewhere
    int best = -1;
    for (size_t i = 0; i < lX.size(); ++i) {
        if (position_of(lX, lX[i]) != int(i) || X.extent[i] < 4 || X.stride[i] <= 0) continue;
        const int inY = position_of(lY, lX[i]), inD = position_of(rq.labelsD, lX[i]);
        if (inY == -2 || inD == -2) continue;
        if (inY < 0 && inD < 0) continue;                      // a label only in this input (Case 4): leave it whole
        if (best < 0 || X.stride[i] > X.stride[size_t(best)]) best = int(i);
    }
    if (best < 0) return;
    hp->idxX = best;
    hp->idxY = position_of(lY, lX[size_t(best)]);
    hp->idxD = position_of(rq.labelsD, lX[size_t(best)]);
    hp->extent = X.extent[size_t(best)];
    hp->strideX = X.stride[size_t(best)];
    hp->strideY = hp->idxY >= 0 ? Y.stride[size_t(hp->idxY)] : 0;
    hp->strideD = hp->idxD >= 0 ? rq.D.stride[size_t(hp->idxD)] : 0;
    // about eight slabs, none below 32 MiB
    int64_t slabs = 8;
    while (slabs > 2 && size_t(std::max(spanA, spanB)) * esz / size_t(slabs) < (size_t(32) << 20)) --slabs;
    hp->slab = (hp->extent + slabs - 1) / slabs;
    if (hp->slab < 1 || hp->slab >= hp->extent) return;
    const int64_t lengths[2] = {hp->slab, hp->extent % hp->slab};
    for (int i = 0; i < 2; ++i) {
        if (lengths[i] == 0) continue;
        btc_contraction_s *sub = new (std::nothrow) btc_contraction_s;
        if (!sub) return;
        hp->sub[i] = sub;
        sub->handle = op->handle;
        sub->req = rq;
        sub->pre_reduce = op->pre_reduce;
        sub->poll_limit = op->poll_limit;
        TensorDesc &sX = hp->slab_is_A ? sub->req.A : sub->req.B, &sY = hp->slab_is_A ? sub->req.B : sub->req.A;
        sX.extent[size_t(hp->idxX)] = lengths[i];
        if (hp->idxY >= 0) sY.extent[size_t(hp->idxY)] = lengths[i];
        if (hp->idxD >= 0) sub->req.D.extent[size_t(hp->idxD)] = lengths[i];
        // a contracted label: later slabs accumulate into D, which needs C's description (= D's)
        sub->req.has_c = true;
        sub->req.C = sub->req.D;
        sub->req.labelsC = sub->req.labelsD;
        sub->req.conjC = rq.has_c ? rq.conjC : false;
        sub->alpha[0] = op->alpha[0]; sub->alpha[1] = op->alpha[1];
        sub->beta[0] = op->beta[0]; sub->beta[1] = op->beta[1];
        if (replan(sub) != BTC_SUCCESS) return;
        span_of_desc(sX, hp->sub_lo[i], hp->sub_hi[i]);
        hp->bytesW = std::max(hp->bytesW, sub->workspace_bytes);
    }
    // slabs of the cut input must not overlap much in memory, or the copies would repeat most of it
    const int64_t slab_span = hp->sub_hi[0] - hp->sub_lo[0] + 1;
    if (double(slab_span) * double((hp->extent + hp->slab - 1) / hp->slab) > 1.25 * double(hp->slab_is_A ? spanA : spanB)) return;
    hp->bytesX = size_t(slab_span) * esz;
    hp->bytesY = size_t(hp->slab_is_A ? spanB : spanA) * esz;
    hp->bytesD = size_t(op->spanD_hi - op->spanD_lo + 1) * esz;
    hp->bytesC = hp->bytesD;
    bool ok = cudaStreamCreateWithFlags(&hp->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    for (int i = 0; i < 2 && ok; ++i) {
        ok = cudaEventCreateWithFlags(&hp->loaded[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaEventCreateWithFlags(&hp->consumed[i], cudaEventDisableTiming) == cudaSuccess &&
             cudaMalloc(reinterpret_cast<void **>(&hp->bufX[i]), hp->bytesX) == cudaSuccess;
    }
    ok = ok && cudaMalloc(reinterpret_cast<void **>(&hp->bufY), hp->bytesY) == cudaSuccess &&
         cudaMalloc(reinterpret_cast<void **>(&hp->bufD), hp->bytesD) == cudaSuccess &&
         (hp->bytesW == 0 || cudaMalloc(reinterpret_cast<void **>(&hp->ws), hp->bytesW) == cudaSuccess);
    if (!ok) { cudaGetLastError(); return; }
    hp->usable = true;
}

// The slabbed run.  X = the cut input, Y = the other one.
btc_error_t run_host_pipeline(btc_contraction_s *op, cudaStream_t st, const void *alpha, const void *A, const void *B,
                              const void *beta, const void *C, void *D, bool use_c)
{
    HostPipeline *hp = op->host;
    const size_t esz = dtype_size(op->plan.dtype);
    const bool c_is_d = use_c && C == D;
    if (use_c && !c_is_d && !hp->bufC && cudaMalloc(reinterpret_cast<void **>(&hp->bufC), hp->bytesC) != cudaSuccess) {
        cudaGetLastError();
        return BTC_ERR_OUT_OF_MEMORY;
    }
    const char *hX = static_cast<const char *>(hp->slab_is_A ? A : B), *hY = static_cast<const char *>(hp->slab_is_A ? B : A);
    const int64_t loY = (hp->slab_is_A ? op->spanB_lo : op->spanA_lo) * int64_t(esz), loD = op->spanD_lo * int64_t(esz);
    bool ok = true;
    auto copy = [&](void *dst, const void *src, size_t n, cudaMemcpyKind kind, cudaStream_t on) {
        ok = ok && cudaMemcpyAsync(dst, src, n, kind, on) == cudaSuccess;
    };
    // the whole of the smaller input, of D's span (padding between its elements must survive the round trip) and of C
    copy(hp->bufY, hY + loY, hp->bytesY, cudaMemcpyHostToDevice, st);
    copy(hp->bufD, static_cast<const char *>(D) + loD, hp->bytesD, cudaMemcpyHostToDevice, st);
    if (use_c && !c_is_d) copy(hp->bufC, static_cast<const char *>(C) + loD, hp->bytesC, cudaMemcpyHostToDevice, st);
    const char *dY = hp->bufY - loY;
    char *dD = hp->bufD - loD;
    const char *dC = use_c ? (c_is_d ? dD : hp->bufC - loD) : nullptr;
    const bool accumulate = hp->idxD < 0;          // a contracted label: slabs add up in D
    const double one[2] = {1.0, 0.0};
    float one_f[2] = {1.f, 0.f};
    const void *beta_one = (op->plan.dtype == BTC_F32 || op->plan.dtype == BTC_C32) ? static_cast<const void *>(one_f) : static_cast<const void *>(one);
    const int64_t count = (hp->extent + hp->slab - 1) / hp->slab;
    // copies run on a stream of their own, one slab ahead of the contraction
    cudaEvent_t start = hp->consumed[0];           // reused below only after its first wait
    ok = ok && cudaEventRecord(start, st) == cudaSuccess && cudaStreamWaitEvent(hp->copy_stream, start, 0) == cudaSuccess;
    btc_error_t rc = BTC_SUCCESS;
    for (int64_t i = 0; i < count && ok && rc == BTC_SUCCESS; ++i) {
        const int b = int(i & 1), which = (i + 1 == count && hp->extent % hp->slab) ? 1 : 0;
        const int64_t first = i * hp->slab;
        const int64_t loX = hp->sub_lo[which] * int64_t(esz);
        const size_t bytes = size_t(hp->sub_hi[which] - hp->sub_lo[which] + 1) * esz;
        if (i >= 2) ok = ok && cudaStreamWaitEvent(hp->copy_stream, hp->consumed[b], 0) == cudaSuccess;
        copy(hp->bufX[b], hX + first * hp->strideX * int64_t(esz) + loX, bytes, cudaMemcpyHostToDevice, hp->copy_stream);
        ok = ok && cudaEventRecord(hp->loaded[b], hp->copy_stream) == cudaSuccess && cudaStreamWaitEvent(st, hp->loaded[b], 0) == cudaSuccess;
        if (!ok) break;
        const char *pX = hp->bufX[b] - loX;
        const char *pY = dY + first * hp->strideY * int64_t(esz);
        char *pD = dD + first * hp->strideD * int64_t(esz);
        const char *pC = dC ? dC + first * hp->strideD * int64_t(esz) : nullptr;
        const void *b_ptr = beta, *c_ptr = pC;
        if (accumulate && i > 0) { b_ptr = beta_one; c_ptr = pD; }     // D += alpha * this slab
        rc = btc_execute(hp->sub[which], st, alpha, hp->slab_is_A ? pX : pY, hp->slab_is_A ? pY : pX, b_ptr, c_ptr, pD,
                         hp->ws, hp->bytesW, nullptr);
        ok = ok && cudaEventRecord(hp->consumed[b], st) == cudaSuccess;
    }
    copy(static_cast<char *>(D) + loD, hp->bufD, hp->bytesD, cudaMemcpyDeviceToHost, st);
    if (cudaStreamSynchronize(st) != cudaSuccess || cudaStreamSynchronize(hp->copy_stream) != cudaSuccess) ok = false;
    if (!ok) { cudaGetLastError(); return rc != BTC_SUCCESS ? rc : BTC_ERR_CUDA; }
    if (rc != BTC_SUCCESS) return rc;
    for (int i = 0; i < 2; ++i)
        for (const btc_contraction_s *o : {static_cast<const btc_contraction_s *>(hp->sub[i]),
                                           static_cast<const btc_contraction_s *>(hp->sub[i] ? hp->sub[i]->real_inner : nullptr)}) {
            if (!o || !o->d_error) continue;
            int32_t word = 0;
            if (cudaMemcpy(&word, o->d_error, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return BTC_ERR_CUDA; }
            if (word != 0) return BTC_ERR_DEVICE_TIMEOUT;
        }
    return BTC_SUCCESS;
}

}  // namespace

extern "C" {

btc_error_t btc_execute_host(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *A,
                             const void *B, const void *beta, const void *C, void *D)
{
    if (!op || !D) return BTC_ERR_INVALID_ARGUMENT;
    if (op->handle.device < 0) return BTC_ERR_CUDA;
    const Plan &pl = op->plan;
    const size_t esz = dtype_size(pl.dtype);
    double al[2] = {op->alpha[0], op->alpha[1]}, be[2] = {op->beta[0], op->beta[1]};
    if (alpha) to_double2(pl.dtype, alpha, al);
    if (beta) to_double2(pl.dtype, beta, be);
    const bool use_ab = !is_zero(al), use_c = !is_zero(be);
    if ((use_ab && (!A || !B)) || (use_c && !C)) return BTC_ERR_INVALID_ARGUMENT;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

    // large inputs: cut the larger one into slabs and copy slab i + 1 while slab i is contracted
    if (use_ab && op->poll_limit == kWaitPollLimit && !pl.mixed) {
        if (!op->host) build_host_pipeline(op);
        if (op->host && op->host->usable) return run_host_pipeline(op, st, alpha, A, B, beta, C, D, use_c);
    }

    struct Buf {
        char *dev = nullptr;
        int64_t lo = 0, hi = 0;
        size_t bytes() const { return size_t(hi - lo + 1); }
    } bA, bB, bC, bD;
    auto span_bytes = [&](Buf &b, int64_t lo, int64_t hi, size_t es) { b.lo = lo * int64_t(es); b.hi = hi * int64_t(es) + int64_t(es) - 1; };
    span_bytes(bA, op->spanA_lo, op->spanA_hi, dtype_size(op->req.A.dtype));
    span_bytes(bB, op->spanB_lo, op->spanB_hi, dtype_size(op->req.B.dtype));
    span_bytes(bD, op->spanD_lo, op->spanD_hi, esz);
    span_bytes(bC, op->spanD_lo, op->spanD_hi, dtype_size(op->req.has_c ? op->req.C.dtype : pl.dtype));
    const bool c_is_d = use_c && C == D;
    void *ws = nullptr;
    btc_error_t rc = BTC_SUCCESS;
    auto fail = [&](btc_error_t e) { if (rc == BTC_SUCCESS) rc = e; };
    auto up = [&](Buf &b, const void *host) {
        if (rc != BTC_SUCCESS) return;
        // 256-byte aligned allocation; the span's first byte keeps the host pointer's offset
        // relative to 16 bytes so that alignment-dependent choices match device-resident use
        if (cudaMalloc(reinterpret_cast<void **>(&b.dev), b.bytes()) != cudaSuccess) { cudaGetLastError(); b.dev = nullptr; fail(BTC_ERR_OUT_OF_MEMORY); return; }
        if (host && cudaMemcpyAsync(b.dev, static_cast<const char *>(host) + b.lo, b.bytes(), cudaMemcpyHostToDevice, st) != cudaSuccess) { cudaGetLastError(); fail(BTC_ERR_CUDA); }
    };
    if (use_ab) { up(bA, A); up(bB, B); }
    up(bD, D);   // D's span travels both ways so that padding between its elements is preserved
    if (use_c && !c_is_d) up(bC, C);
    if (rc == BTC_SUCCESS && op->workspace_bytes > 0 &&
        cudaMalloc(&ws, op->workspace_bytes) != cudaSuccess) { cudaGetLastError(); ws = nullptr; fail(BTC_ERR_OUT_OF_MEMORY); }
    if (rc == BTC_SUCCESS) {
        const void *dA = use_ab ? bA.dev - bA.lo : nullptr, *dB = use_ab ? bB.dev - bB.lo : nullptr;
        void *dD = bD.dev - bD.lo;
        const void *dC = use_c ? (c_is_d ? dD : static_cast<void *>(bC.dev - bC.lo)) : nullptr;
        rc = btc_execute(op, cuda_stream, alpha, dA, dB, beta, dC, dD, ws, op->workspace_bytes, nullptr);
    }
    if (rc == BTC_SUCCESS &&
        cudaMemcpyAsync(static_cast<char *>(D) + bD.lo, bD.dev, bD.bytes(), cudaMemcpyDeviceToHost, st) != cudaSuccess) { cudaGetLastError(); fail(BTC_ERR_CUDA); }
    if (cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); fail(BTC_ERR_CUDA); }
    // a bounded device-side wait that gave up left D incomplete: say so
    for (const btc_contraction_s *o : {static_cast<const btc_contraction_s *>(op), static_cast<const btc_contraction_s *>(op->real_inner)}) {
        if (rc != BTC_SUCCESS || !o || !o->d_error) continue;
        int32_t word = 0;
        if (cudaMemcpy(&word, o->d_error, sizeof word, cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); fail(BTC_ERR_CUDA); }
        else if (word != 0) fail(BTC_ERR_DEVICE_TIMEOUT);
    }
    for (Buf *b : {&bA, &bB, &bD}) if (b->dev) cudaFree(b->dev);
    if (use_c && !c_is_d && bC.dev) cudaFree(bC.dev);
    if (ws) cudaFree(ws);
    return rc;
}


// ---- execute without any allocation -------------------------------------------------------------
// Scratch for split-K partial sums that belongs to the library image itself: every GPU that loads
// the library holds these bytes until the process exits.
#define BTC_STATIC_SCRATCH_BYTES (8u << 20)
static __device__ __align__(256) unsigned char btc_static_scratch[BTC_STATIC_SCRATCH_BYTES];

btc_error_t btc_execute_static_scratch(btc_contraction_t op, void *cuda_stream, const void *alpha, const void *A,
                                       const void *B, const void *beta, const void *C, void *D)
{
    // Device address of the array, looked up once per device.  In host code the array's name is
    // only a stand-in for the symbol, never an address a kernel could use.
    static std::atomic<void *> scratch_of_device[64] = {};
    if (!op || !D) return BTC_ERR_INVALID_ARGUMENT;
    if (op->handle.device < 0) return BTC_ERR_CUDA;
    if (op->workspace_floor > size_t(BTC_STATIC_SCRATCH_BYTES)) return BTC_ERR_SCRATCH_LIMIT;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return BTC_ERR_CUDA; }
    // the symbol's address differs per device: the operation's device must be the current one
    if (dev != op->handle.device || dev < 0 || dev >= 64) return BTC_ERR_INVALID_ARGUMENT;
    void *scratch = scratch_of_device[dev].load(std::memory_order_relaxed);
    if (!scratch) {
        if (cudaGetSymbolAddress(&scratch, btc_static_scratch) != cudaSuccess || !scratch) {
            cudaGetLastError();
            return BTC_ERR_CUDA;
        }
        scratch_of_device[dev].store(scratch, std::memory_order_relaxed);   // racing first calls store the same value
    }
    // Every consumer thread of every CTA overwrites all of its partial sums before the reduction
    // kernel reads them, so nothing in the array has to start at zero.
    return btc_execute(op, cuda_stream, alpha, A, B, beta, C, D, scratch, size_t(BTC_STATIC_SCRATCH_BYTES), nullptr);
}

// ---- binary / unary operation -------------------------------------------------------------------
btc_error_t btc_create_elementwise(btc_handle_t handle, btc_tensor_info_t A, const int64_t *labelsA, int conjA,
                                   btc_tensor_info_t B, int conjB, btc_tensor_info_t C, const int64_t *labelsC,
                                   const void *alpha, const void *beta, btc_elementwise_t *out)
{
    if (!handle || !A || !C || !out) return BTC_ERR_INVALID_ARGUMENT;
    if ((!labelsA && !A->desc.extent.empty()) || (!labelsC && !C->desc.extent.empty())) return BTC_ERR_INVALID_ARGUMENT;
    btc_elementwise_s *op = new (std::nothrow) btc_elementwise_s;
    if (!op) return BTC_ERR_OUT_OF_MEMORY;
    op->handle = *handle;
    op->req.A = A->desc;
    op->req.C = C->desc;
    op->req.has_b = B != nullptr;
    if (B) op->req.B = B->desc;
    op->req.labelsA.assign(labelsA, labelsA + A->desc.extent.size());
    op->req.labelsC.assign(labelsC, labelsC + C->desc.extent.size());
    op->req.conjA = conjA != 0;
    op->req.conjB = conjB != 0;
    if (alpha) to_double2(C->desc.dtype, alpha, op->alpha);
    if (beta) to_double2(C->desc.dtype, beta, op->beta);
    int rc = (!B && !is_zero(op->beta)) ? int(BTC_ERR_INVALID_ARGUMENT) : make_elementwise_plan(op->req, op->plan);
    if (rc == BTC_SUCCESS && (op->plan.keep.size() > size_t(kGenericMaxD) || op->plan.sum.size() > size_t(kGenericMaxD)))
        rc = BTC_ERR_NOT_SUPPORTED;
    if (rc != BTC_SUCCESS) {
        delete op;
        return btc_error_t(rc);
    }
    *out = op;
    return BTC_SUCCESS;
}

btc_error_t btc_destroy_elementwise(btc_elementwise_t *op)
{
    if (!op) return BTC_ERR_INVALID_ARGUMENT;
    delete *op;
    *op = nullptr;
    return BTC_SUCCESS;
}

btc_error_t btc_elementwise_get_attr(btc_elementwise_t op, int32_t key, void *value, size_t len, size_t *needed)
{
    if (!op) return BTC_ERR_INVALID_ARGUMENT;
    int32_t i32[2];
    size_t n = 0;
    switch (key) {
    case BTC_EW_ATTR_KERNEL: i32[0] = int32_t(op->plan.kernel); n = 4; break;
    case BTC_EW_ATTR_LAST_KERNEL: i32[0] = op->last_kernel; n = 4; break;
    case BTC_EW_ATTR_NUM_MODES: i32[0] = int32_t(op->plan.keep.size()); i32[1] = int32_t(op->plan.sum.size()); n = 8; break;
    default: return BTC_ERR_INVALID_ARGUMENT;
    }
    if (needed) *needed = n;
    if (!value) return needed ? BTC_SUCCESS : BTC_ERR_INVALID_ARGUMENT;
    if (len < n) return BTC_ERR_INVALID_ARGUMENT;
    std::memcpy(value, i32, n);
    return BTC_SUCCESS;
}

btc_error_t btc_elementwise_execute(btc_elementwise_t op, void *cuda_stream, const void *alpha, const void *A,
                                    const void *beta, const void *B, void *C)
{
    if (!op || !C) return BTC_ERR_INVALID_ARGUMENT;
    if (op->handle.device < 0) return BTC_ERR_CUDA;
    const ElementwisePlan &pl = op->plan;
    double al[2] = {op->alpha[0], op->alpha[1]}, be[2] = {op->beta[0], op->beta[1]};
    if (alpha) to_double2(pl.dtype, alpha, al);
    if (beta) to_double2(pl.dtype, beta, be);
    const bool use_a = !is_zero(al), use_b = !is_zero(be);
    if ((use_a && !A) || (use_b && (!B || !pl.has_b))) return BTC_ERR_INVALID_ARGUMENT;
    const size_t part = dtype_is_complex(pl.dtype) ? dtype_size(pl.dtype) / 2 : dtype_size(pl.dtype);
    auto misaligned = [&](const void *q) { return q && (reinterpret_cast<uintptr_t>(q) % part) != 0; };
    if (misaligned(A) || misaligned(B) || misaligned(C)) return BTC_ERR_MISALIGNED;
    ElementwiseParams p;
    std::memset(&p, 0, sizeof p);
    p.A = A; p.B = B; p.C = C;
    p.nk = int32_t(pl.keep.size()); p.ns = int32_t(pl.sum.size());
    p.total_keep = pl.total_keep; p.total_sum = pl.total_sum;
    for (int i = 0; i < p.nk; ++i) {
        const Mode &m = pl.keep[size_t(i)];
        p.ext_k[i] = m.extent; p.sA_k[i] = m.sA; p.sB_k[i] = m.sB; p.sC_k[i] = m.sD;
    }
    {
        auto reciprocal = [](int64_t ext, uint32_t &mul, uint32_t &shift) {
            int s = 0;
            while ((int64_t(1) << s) < ext) ++s;
            shift = uint32_t(31 + s);
            mul = uint32_t(((uint64_t(1) << shift) + uint64_t(ext) - 1) / uint64_t(ext));
        };
        const int64_t vlen = int64_t(16 / dtype_size(pl.dtype));
        for (int i = 0; i < p.nk; ++i)
            if (p.ext_k[i] < (int64_t(1) << 31)) reciprocal(p.ext_k[i], p.div_mul[i], p.div_shift[i]);
        if (p.nk > 0 && vlen > 0 && p.ext_k[0] % vlen == 0 && p.ext_k[0] < (int64_t(1) << 31))
            reciprocal(p.ext_k[0] / vlen, p.div_mul[kGenericMaxD], p.div_shift[kGenericMaxD]);
    }
    int64_t min_sum = INT64_MAX, min_keep = INT64_MAX;
    for (int i = 0; i < p.ns; ++i) {
        p.ext_s[i] = pl.sum[size_t(i)].extent; p.sA_s[i] = pl.sum[size_t(i)].sA;
        min_sum = std::min<int64_t>(min_sum, std::llabs(p.sA_s[i]));
    }
    for (int i = 0; i < p.nk; ++i)
        if (p.sA_k[i] != 0) min_keep = std::min<int64_t>(min_keep, std::llabs(p.sA_k[i]));
    p.alpha[0] = al[0]; p.alpha[1] = al[1]; p.beta[0] = be[0]; p.beta[1] = be[1];
    p.conjA = pl.conjA; p.conjB = pl.conjB;
    p.use_a = use_a; p.use_b = use_b;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    const bool narrow = pl.total_keep < (int64_t(1) << 31) && pl.total_sum < (int64_t(1) << 31);
    const bool transposing = pl.kernel == ElementwiseKernel::TRANSPOSING && use_a;
#define BTC_EW_TRANSPOSE(R, CPLX, I, SUMS, WHEN, FLAGS)                                                            \
    if (WHEN) {                                                                                                    \
        if (set_smem_once(elementwise_transposing_kernel<R, CPLX, I, SUMS>, TT::SMEM_BYTES, FLAGS) != cudaSuccess) return BTC_ERR_CUDA; \
        elementwise_transposing_kernel<R, CPLX, I, SUMS><<<unsigned(blocks), TT::THREADS, TT::SMEM_BYTES, st>>>(p); \
    }
#define BTC_EW_LAUNCH(R, CPLX)                                                                                     \
    do {                                                                                                           \
        if (transposing) {                                                                                         \
            typedef TransposeTile<R, CPLX> TT;                                                                     \
            static std::atomic<bool> configured[4][64] = {};                                                       \
            BTC_EW_TRANSPOSE(R, CPLX, uint32_t, false, narrow && p.ns == 0, configured[0]);                        \
            BTC_EW_TRANSPOSE(R, CPLX, uint32_t, true, narrow && p.ns != 0, configured[1]);                         \
            BTC_EW_TRANSPOSE(R, CPLX, int64_t, false, !narrow && p.ns == 0, configured[2]);                        \
            BTC_EW_TRANSPOSE(R, CPLX, int64_t, true, !narrow && p.ns != 0, configured[3]);                         \
        } else if (lanes == 32) {                                                                                  \
            if (narrow) elementwise_direct_kernel<R, CPLX, 32, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);      \
            else elementwise_direct_kernel<R, CPLX, 32, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);              \
        } else {                                                                                                   \
            if (narrow) elementwise_direct_kernel<R, CPLX, 1, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);       \
            else elementwise_direct_kernel<R, CPLX, 1, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);               \
        }                                                                                                          \
    } while (0)
    int lanes = 1;
    int64_t blocks = 1;
    // 16-byte vectors along dimension 0 when nothing is summed and that dimension is contiguous in
    // every tensor in use, with all other strides and the base pointers keeping 16-byte alignment
    const int vec = int(16 / dtype_size(pl.dtype));
    bool vector_ok = !transposing && p.ns == 0 && p.nk >= 1 && vec > 1 && p.ext_k[0] % vec == 0 && p.sC_k[0] == 1 &&
                     (!use_a || p.sA_k[0] == 1) && (!use_b || p.sB_k[0] == 1) &&
                     reinterpret_cast<uintptr_t>(C) % 16 == 0 && (!use_a || reinterpret_cast<uintptr_t>(A) % 16 == 0) &&
                     (!use_b || reinterpret_cast<uintptr_t>(B) % 16 == 0);
    for (int i = 1; vector_ok && i < p.nk; ++i)
        vector_ok = p.sC_k[i] % vec == 0 && (!use_a || p.sA_k[i] % vec == 0) && (!use_b || p.sB_k[i] % vec == 0);
    op->last_kernel = vector_ok ? 3 : (transposing ? 2 : 1);
    if (vector_ok) {
        blocks = (pl.total_keep / vec + 255) / 256;
        const int64_t cap = int64_t(op->handle.sm_count) * 32;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
        switch (pl.dtype) {
        case BTC_F32:
            if (narrow) elementwise_vector_kernel<float, false, 4, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);
            else elementwise_vector_kernel<float, false, 4, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);
            break;
        case BTC_F64:
            if (narrow) elementwise_vector_kernel<double, false, 2, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);
            else elementwise_vector_kernel<double, false, 2, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);
            break;
        default:   // complex64: two elements per 16 bytes (complex128 has vec == 1)
            if (narrow) elementwise_vector_kernel<float, true, 2, uint32_t><<<unsigned(blocks), 256, 0, st>>>(p);
            else elementwise_vector_kernel<float, true, 2, int64_t><<<unsigned(blocks), 256, 0, st>>>(p);
            break;
        }
        return cudaGetLastError() == cudaSuccess ? BTC_SUCCESS : BTC_ERR_CUDA;
    }
    if (transposing) {
        const int T = dtype_size(pl.dtype) <= 8 ? 64 : 32;
        const int TC = dtype_size(pl.dtype) == 4 ? TransposeTile<float, false>::TC : T;
        const int TA = dtype_size(pl.dtype) == 4 ? TransposeTile<float, false>::TA : T;
        p.tile_mode_a = pl.tile_mode_a;
        p.tiles_c = int32_t((p.ext_k[0] + TC - 1) / TC);
        p.tiles_a = int32_t((p.ext_k[pl.tile_mode_a] + TA - 1) / TA);
        p.rest = pl.total_keep / (p.ext_k[0] * p.ext_k[pl.tile_mode_a]);
        blocks = int64_t(p.tiles_c) * p.tiles_a * p.rest;
        if (blocks > 0x7fffffffLL) return BTC_ERR_NOT_SUPPORTED;
    } else {
        lanes = (use_a && p.ns > 0 && min_sum < min_keep && pl.total_sum >= 32) ? 32 : 1;
        blocks = (pl.total_keep * lanes + 255) / 256;
        const int64_t cap = int64_t(op->handle.sm_count) * 32;
        if (blocks > cap) blocks = cap;
        if (blocks < 1) blocks = 1;
    }
    switch (pl.dtype) {
    case BTC_F32: BTC_EW_LAUNCH(float, false); break;
    case BTC_F64: BTC_EW_LAUNCH(double, false); break;
    case BTC_C32: BTC_EW_LAUNCH(float, true); break;
    default: BTC_EW_LAUNCH(double, true); break;
    }
#undef BTC_EW_LAUNCH
#undef BTC_EW_TRANSPOSE
    return cudaGetLastError() == cudaSuccess ? BTC_SUCCESS : BTC_ERR_CUDA;
}

btc_error_t btc_selftest_bounded_wait(btc_handle_t handle, void *cuda_stream, int32_t polls, int32_t *error_code,
                                      int32_t *threads_gave_up)
{
    if (!handle || !error_code || !threads_gave_up || polls < 1 || polls > 65536) return BTC_ERR_INVALID_ARGUMENT;
    if (handle->device < 0) return BTC_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int *words = nullptr;
    if (cudaMalloc(reinterpret_cast<void **>(&words), 2 * sizeof(int)) != cudaSuccess) { cudaGetLastError(); return BTC_ERR_OUT_OF_MEMORY; }
    btc_error_t rc = BTC_SUCCESS;
    int host[2] = {0, 0};
    if (cudaMemsetAsync(words, 0, 2 * sizeof(int), st) != cudaSuccess) rc = BTC_ERR_CUDA;
    if (rc == BTC_SUCCESS) {
        bounded_wait_selftest_kernel<0><<<1, 64, 0, st>>>(unsigned(polls), words, words + 1);
        if (cudaGetLastError() != cudaSuccess) rc = BTC_ERR_CUDA;
    }
    if (rc == BTC_SUCCESS && (cudaMemcpyAsync(host, words, sizeof host, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                              cudaStreamSynchronize(st) != cudaSuccess)) { cudaGetLastError(); rc = BTC_ERR_CUDA; }
    cudaFree(words);
    *error_code = host[0];
    *threads_gave_up = host[1];
    return rc;
}

btc_error_t btc_status_get(btc_status_t status, int32_t key, void *value, size_t len)
{
    if (!status || !value) return BTC_ERR_INVALID_ARGUMENT;
    switch (key) {
    case BTC_STATUS_KERNEL: if (len < 4) return BTC_ERR_INVALID_ARGUMENT; std::memcpy(value, &status->kernel, 4); break;
    case BTC_STATUS_LAUNCHES: if (len < 4) return BTC_ERR_INVALID_ARGUMENT; std::memcpy(value, &status->launches, 4); break;
    case BTC_STATUS_GRID: if (len < 12) return BTC_ERR_INVALID_ARGUMENT; std::memcpy(value, status->grid, 12); break;
    case BTC_STATUS_SPLIT_K: if (len < 4) return BTC_ERR_INVALID_ARGUMENT; std::memcpy(value, &status->split_k, 4); break;
    case BTC_STATUS_VARIANT: if (len < 4) return BTC_ERR_INVALID_ARGUMENT; std::memcpy(value, &status->variant, 4); break;
    default: return BTC_ERR_INVALID_ARGUMENT;
    }
    return BTC_SUCCESS;
}

btc_error_t btc_destroy_status(btc_status_t *status)
{
    if (!status) return BTC_ERR_INVALID_ARGUMENT;
    delete *status;
    *status = nullptr;
    return BTC_SUCCESS;
}

btc_error_t btc_explain_error(btc_error_t code, char *buf, size_t len, size_t *needed)
{
    const char *msg = "unknown error code";
    switch (code) {
    case BTC_SUCCESS: msg = "success"; break;
    case BTC_ERR_INVALID_ARGUMENT: msg = "invalid argument (NULL where a value is required, bad rank, key or enum)"; break;
    case BTC_ERR_INVALID_EXTENT: msg = "an extent is smaller than 1"; break;
    case BTC_ERR_EXTENT_MISMATCH: msg = "modes that share a label have different extents"; break;
    case BTC_ERR_C_D_MISMATCH: msg = "C does not have D's rank, extents, strides and labels"; break;
    case BTC_ERR_D_ALIASING: msg = "two index tuples of D address the same element"; break;
    case BTC_ERR_LABEL_ONLY_IN_D: msg = "a label of D occurs in neither A nor B"; break;
    case BTC_ERR_NOT_SUPPORTED: msg = "operation not supported (mixed element types, label repeated inside D, or size limits)"; break;
    case BTC_ERR_WORKSPACE_TOO_SMALL: msg = "workspace missing or smaller than btc_contraction_workspace_size"; break;
    case BTC_ERR_MISALIGNED: msg = "a data pointer is not aligned to its element size (workspace: 256 bytes)"; break;
    case BTC_ERR_CUDA: msg = "a CUDA runtime call failed or no CUDA device is available"; break;
    case BTC_ERR_DEVICE_TIMEOUT: msg = "a bounded device-side wait expired"; break;
    case BTC_ERR_OUT_OF_MEMORY: msg = "out of memory"; break;
    case BTC_ERR_SCRATCH_LIMIT: msg = "the operation needs more scratch than the library's built-in 8 MiB array; use btc_execute with a caller-provided workspace"; break;
    default: break;
    }
    const size_t n = std::strlen(msg) + 1;
    if (needed) *needed = n;
    if (buf && len > 0) {
        const size_t c = n < len ? n : len;
        std::memcpy(buf, msg, c);
        buf[c - 1] = '\0';
    }
    return BTC_SUCCESS;
}

}  // extern "C"

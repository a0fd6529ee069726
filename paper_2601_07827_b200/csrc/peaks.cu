// Peak micro-benchmarks: what this GPU's arithmetic pipes and its memory sustain, measured with
// kernels that do nothing else, so that a roofline fraction can be quoted against a number taken
// on the same device in the same run (btc_measure_peak in include/btc.h).
//   arithmetic: register-resident loops of independent FMA / MMA chains (no memory traffic);
//               the count is the flops the loop executes, the time a pair of CUDA events.
//   memory:     one pass over a caller-provided buffer: read-only (sum), write-only (fill),
//               copy (first half to second half), 16-byte accesses, grid-stride.
#include <cuda_runtime.h>

#include <cstdint>

#include "../../include/btc.h"

namespace {

constexpr int kThreads = 256;
__device__ double g_sink;                // target of stores that never happen: keeps the loops alive

template <typename T> __device__ __forceinline__ T fma_t(T a, T b, T c);
template <> __device__ __forceinline__ float fma_t<float>(float a, float b, float c) { return fmaf(a, b, c); }
template <> __device__ __forceinline__ double fma_t<double>(double a, double b, double c) { return fma(a, b, c); }

// 16 independent FMA chains per thread
template <typename T>
__global__ void __launch_bounds__(kThreads) fma_loop_kernel(int iters, T seed)
{
    T acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = seed + T(i + threadIdx.x);
    const T a = seed * T(0.5), b = seed * T(0.25);
#pragma unroll 8
    for (int it = 0; it < iters; ++it)
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = fma_t<T>(acc[i], a, b);
    T s = T(0);
#pragma unroll
    for (int i = 0; i < 16; ++i) s += acc[i];
    if (s == T(123456789)) g_sink = double(s);      // never true
}

// FP64 tensor-core MMAs, 8 independent accumulator fragments per warp
template <bool K16>
__global__ void __launch_bounds__(kThreads) dmma_loop_kernel(int iters, double seed)
{
    double c[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = seed + i + j;
    double a[8], b[4];
#pragma unroll
    for (int j = 0; j < 8; ++j) a[j] = seed * (j + 1);
#pragma unroll
    for (int j = 0; j < 4; ++j) b[j] = seed / (j + 1);
#pragma unroll 1
    for (int it = 0; it < iters; ++it)
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            if (K16)
                asm volatile("mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
                             "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
                             : "+d"(c[i][0]), "+d"(c[i][1]), "+d"(c[i][2]), "+d"(c[i][3])
                             : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(a[4]), "d"(a[5]), "d"(a[6]), "d"(a[7]),
                               "d"(b[0]), "d"(b[1]), "d"(b[2]), "d"(b[3]));
            else
                asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                             : "+d"(c[i][0]), "+d"(c[i][1]) : "d"(a[0]), "d"(b[0]));
        }
    double s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += c[i][0] + c[i][1] + c[i][2] + c[i][3];
    if (s == 123456789.0) g_sink = s;
}

// TF32 tensor-core MMAs through the warp-level instruction (m16n8k8), 8 independent fragments
__global__ void __launch_bounds__(kThreads) tf32_mma_loop_kernel(int iters, float seed)
{
    float c[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) c[i][j] = seed + i + j;
    unsigned a[4], b[2];
#pragma unroll
    for (int j = 0; j < 4; ++j) a[j] = __float_as_uint(seed * (j + 1)) & 0xffffe000u;
    b[0] = __float_as_uint(seed) & 0xffffe000u; b[1] = __float_as_uint(seed * 0.5f) & 0xffffe000u;
#pragma unroll 1
    for (int it = 0; it < iters; ++it)
#pragma unroll
        for (int i = 0; i < 8; ++i)
            asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                         : "+f"(c[i][0]), "+f"(c[i][1]), "+f"(c[i][2]), "+f"(c[i][3])
                         : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
    float s = 0;
#pragma unroll
    for (int i = 0; i < 8; ++i) s += c[i][0] + c[i][1] + c[i][2] + c[i][3];
    if (s == 123456789.f) g_sink = s;
}

__global__ void __launch_bounds__(kThreads) hbm_read_kernel(const float4 *src, size_t n)
{
    float s = 0.f;
    const size_t stride = size_t(gridDim.x) * kThreads;
    size_t i = size_t(blockIdx.x) * kThreads + threadIdx.x;
    for (; i + 3 * stride < n; i += 4 * stride) {        // four loads in flight per thread
        const float4 a = src[i], b = src[i + stride], c = src[i + 2 * stride], d = src[i + 3 * stride];
        s += a.x + b.y + c.z + d.w;
    }
    for (; i < n; i += stride) s += src[i].x;
    if (s == 123456789.f) g_sink = s;
}

__global__ void __launch_bounds__(kThreads) hbm_write_kernel(float4 *dst, size_t n, float value)
{
    const float4 v = make_float4(value, value, value, value);
    const size_t stride = size_t(gridDim.x) * kThreads;
    for (size_t i = size_t(blockIdx.x) * kThreads + threadIdx.x; i < n; i += stride) dst[i] = v;
}

__global__ void __launch_bounds__(kThreads) hbm_copy_kernel(const float4 *src, float4 *dst, size_t n)
{
    const size_t stride = size_t(gridDim.x) * kThreads;
    size_t i = size_t(blockIdx.x) * kThreads + threadIdx.x;
    for (; i + 7 * stride < n; i += 8 * stride) {         // eight loads in flight per thread
        float4 v[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) v[j] = __ldcs(src + i + j * stride);
#pragma unroll
        for (int j = 0; j < 8; ++j) __stcs(dst + i + j * stride, v[j]);
    }
    for (; i < n; i += stride) dst[i] = src[i];
}

}  // namespace

extern "C" btc_error_t btc_measure_peak(btc_handle_t handle, int32_t which, void *cuda_stream, void *buffer, size_t bytes,
                                        int32_t repeats, double *value)
{
    if (!handle || !value || repeats < 1) return BTC_ERR_INVALID_ARGUMENT;
    int dev = -1, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) {
        cudaGetLastError();
        return BTC_ERR_CUDA;
    }
    const bool memory = which >= BTC_PEAK_HBM_READ && which <= BTC_PEAK_HBM_COPY;
    if (which < BTC_PEAK_FP64_FMA || which > BTC_PEAK_HBM_COPY) return BTC_ERR_INVALID_ARGUMENT;
    if (memory && (!buffer || bytes < (size_t(1) << 20) || reinterpret_cast<uintptr_t>(buffer) % 16)) return BTC_ERR_INVALID_ARGUMENT;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaEvent_t e0, e1;
    if (cudaEventCreate(&e0) != cudaSuccess || cudaEventCreate(&e1) != cudaSuccess) { cudaGetLastError(); return BTC_ERR_CUDA; }
    const int iters = 4096;
    const int grid = sms * 8;                       // 8 CTAs of 256 threads per SM (one wave)
    double work = 0.0;                              // flops or bytes per launch
    for (int r = -1; r < repeats; ++r) {            // one warm-up launch, then the timed ones
        if (r == 0) cudaEventRecord(e0, st);
        switch (which) {
        case BTC_PEAK_FP64_FMA:
            fma_loop_kernel<double><<<grid, kThreads, 0, st>>>(iters, 1.0000001);
            work = 2.0 * 16 * iters * double(grid) * kThreads;
            break;
        case BTC_PEAK_FP32_FMA:
            fma_loop_kernel<float><<<grid, kThreads, 0, st>>>(iters, 1.0000001f);
            work = 2.0 * 16 * iters * double(grid) * kThreads;
            break;
        case BTC_PEAK_FP64_MMA_K16:
            dmma_loop_kernel<true><<<grid, kThreads, 0, st>>>(iters, 1.0000001);
            work = 2.0 * 16 * 8 * 16 * 8.0 * iters * double(grid) * (kThreads / 32);
            break;
        case BTC_PEAK_FP64_MMA_K4:
            dmma_loop_kernel<false><<<grid, kThreads, 0, st>>>(iters, 1.0000001);
            work = 2.0 * 8 * 8 * 4 * 8.0 * iters * double(grid) * (kThreads / 32);
            break;
        case BTC_PEAK_TF32_MMA_SYNC:
            tf32_mma_loop_kernel<<<grid, kThreads, 0, st>>>(iters, 1.0000001f);
            work = 2.0 * 16 * 8 * 8 * 8.0 * iters * double(grid) * (kThreads / 32);
            break;
        case BTC_PEAK_HBM_READ:
            hbm_read_kernel<<<grid, kThreads, 0, st>>>(static_cast<const float4 *>(buffer), bytes / 16);
            work = double(bytes / 16 * 16);
            break;
        case BTC_PEAK_HBM_WRITE:
            hbm_write_kernel<<<grid, kThreads, 0, st>>>(static_cast<float4 *>(buffer), bytes / 16, 1.0f);
            work = double(bytes / 16 * 16);
            break;
        default: {
            const size_t half = bytes / 32;         // 16-byte elements in each half
            hbm_copy_kernel<<<grid, kThreads, 0, st>>>(static_cast<const float4 *>(buffer), static_cast<float4 *>(buffer) + half, half);
            work = 2.0 * double(half * 16);         // bytes read + bytes written
        } break;
        }
    }
    btc_error_t rc = BTC_SUCCESS;
    float ms = 0.f;
    if (cudaEventRecord(e1, st) != cudaSuccess || cudaEventSynchronize(e1) != cudaSuccess || cudaGetLastError() != cudaSuccess ||
        cudaEventElapsedTime(&ms, e0, e1) != cudaSuccess || ms <= 0.f) {
        cudaGetLastError();
        rc = BTC_ERR_CUDA;
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    if (rc == BTC_SUCCESS) *value = work * repeats / (double(ms) * 1e-3);      // flop/s or byte/s
    return rc;
}

// C := alpha op(A) + beta op(B)  (Sec. "Unary and Binary Operations"): labels only in A are summed
// over, A is broadcast along labels only in C, repeated labels of A act through summed strides.
// Both kernels are bandwidth-bound passes: A (and B) read once through their strides, C written
// once through its own.
//   direct       one thread (or one warp, lanes over the summed index) per element of C, C's
//                most contiguous dimension fastest.  Right when A is contiguous along the same
//                dimension (scaling, addition, reduction, broadcast).
//   transposing  permutations whose input is contiguous along another dimension than the output:
//                a CTA moves a 32 x 32 tile through shared memory, reading along A's dimension and
//                writing along C's, so both sides see whole 128-byte lines.
// Sums are kept in double (pairs for complex) for every element type.
#pragma once

#include <cuda_runtime.h>

#include "isolated_sum_kernel.cuh"
#include "kernel_params.h"

namespace btc {

// alpha * (acc_r, acc_i) + beta * op(b) -> C[off]
template <typename R, bool CPLX>
__device__ __forceinline__ void elementwise_finish(const ElementwiseParams &p, int64_t offB, int64_t offC, double acc_r, double acc_i)
{
    constexpr int NC = CPLX ? 2 : 1;
    R *C = static_cast<R *>(p.C);
    double c_r = p.alpha[0] * acc_r - p.alpha[1] * acc_i;
    double c_i = p.alpha[0] * acc_i + p.alpha[1] * acc_r;
    if (p.use_b) {
        const R *B = static_cast<const R *>(p.B);
        const double br = double(B[NC * offB]);
        const double bi = CPLX ? (p.conjB ? -double(B[NC * offB + (NC - 1)]) : double(B[NC * offB + (NC - 1)])) : 0.0;
        c_r += p.beta[0] * br - p.beta[1] * bi;
        c_i += p.beta[0] * bi + p.beta[1] * br;
    }
    C[NC * offC] = R(c_r);
    if (CPLX) C[NC * offC + (NC - 1)] = R(c_i);
}

// sum over the summed dimensions of A starting at element offset `base`; lanes stride over the
// summed index when LANES > 1 (the caller reduces across lanes)
template <typename R, bool CPLX, int LANES, typename I>
__device__ __forceinline__ void elementwise_sum(const ElementwiseParams &p, int64_t base, int lane, double &acc_r, double &acc_i)
{
    constexpr int NC = CPLX ? 2 : 1;
    constexpr int U = 4;
    const R *A = static_cast<const R *>(p.A);
    acc_r = acc_i = 0.0;
    if (!p.use_a) return;
    if (p.ns == 0) {                       // nothing to sum: one element
        if (lane == 0) {
            acc_r = double(A[NC * base]);
            if (CPLX) acc_i = double(A[NC * base + (NC - 1)]);
        }
    } else {
        for (int64_t s0 = lane; s0 < p.total_sum; s0 += int64_t(U) * LANES) {
            R v_r[U], v_i[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t s = s0 + int64_t(u) * LANES;
                const bool in = s < p.total_sum;
                const int64_t off = base + (in ? decode_offset<I>(I(s), p.ns, p.ext_s, p.sA_s) : 0);
                v_r[u] = in ? A[NC * off] : R(0);
                v_i[u] = (CPLX && in) ? A[NC * off + (NC - 1)] : R(0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                acc_r += double(v_r[u]);
                if (CPLX) acc_i += double(v_i[u]);
            }
        }
    }
    if (CPLX && p.conjA) acc_i = -acc_i;   // conjugation commutes with the sum
}

template <typename R, bool CPLX, int LANES, typename I>
__global__ void __launch_bounds__(256) elementwise_direct_kernel(const ElementwiseParams p)
{
    const int lane = (LANES == 1) ? 0 : int(threadIdx.x) % LANES;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) / LANES;
    const int64_t ngroups = (int64_t(gridDim.x) * blockDim.x) / LANES;
    for (int64_t e = group; e < p.total_keep; e += ngroups) {
        int64_t offA = 0, offB = 0, offC = 0;
        I lin = I(e);
        for (int d = 0; d < p.nk; ++d) {
            const I ext = I(p.ext_k[d]);
            const I q = lin / ext;
            const int64_t i = int64_t(lin - q * ext);
            lin = q;
            offA += i * p.sA_k[d];
            offB += i * p.sB_k[d];
            offC += i * p.sC_k[d];
        }
        double acc_r, acc_i;
        elementwise_sum<R, CPLX, LANES, I>(p, offA, lane, acc_r, acc_i);
        if (LANES > 1) {
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) {
                acc_r += __shfl_xor_sync(0xffffffffu, acc_r, o);
                if (CPLX) acc_i += __shfl_xor_sync(0xffffffffu, acc_i, o);
            }
        }
        if (lane == 0) elementwise_finish<R, CPLX>(p, offB, offC, acc_r, acc_i);
    }
}

// blockIdx.x enumerates (tile along C's dimension 0, tile along A's dimension, rest), first fastest;
// 32 x 8 threads, each 4 elements of the 32 x 32 tile in either phase
template <typename R, bool CPLX, typename I>
__global__ void __launch_bounds__(256) elementwise_transposing_kernel(const ElementwiseParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    __shared__ double tile[NC][32][33];
    const int ma = p.tile_mode_a;
    const int64_t tile_c = blockIdx.x % p.tiles_c;
    const int64_t tile_a = (blockIdx.x / p.tiles_c) % p.tiles_a;
    int64_t lin = blockIdx.x / (int64_t(p.tiles_c) * p.tiles_a);
    int64_t restA = 0, restB = 0, restC = 0;
    for (int d = 1; d < p.nk; ++d) {
        if (d == ma) continue;
        const int64_t i = lin % p.ext_k[d];
        lin /= p.ext_k[d];
        restA += i * p.sA_k[d];
        restB += i * p.sB_k[d];
        restC += i * p.sC_k[d];
    }
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int64_t c0 = tile_c * 32, a0 = tile_a * 32;
    const int64_t ext_c = p.ext_k[0], ext_a = p.ext_k[ma];
    // phase 1: consecutive threads along A's dimension
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int64_t c = c0 + ty + 8 * r, a = a0 + tx;
        double acc_r = 0.0, acc_i = 0.0;
        if (c < ext_c && a < ext_a)
            elementwise_sum<R, CPLX, 1, I>(p, restA + c * p.sA_k[0] + a * p.sA_k[ma], 0, acc_r, acc_i);
        tile[0][ty + 8 * r][tx] = acc_r;
        if (CPLX) tile[NC - 1][ty + 8 * r][tx] = acc_i;
    }
    __syncthreads();
    // phase 2: consecutive threads along C's dimension 0
#pragma unroll
    for (int r = 0; r < 4; ++r) {
        const int64_t c = c0 + tx, a = a0 + ty + 8 * r;
        if (c < ext_c && a < ext_a)
            elementwise_finish<R, CPLX>(p, restB + c * p.sB_k[0] + a * p.sB_k[ma], restC + c * p.sC_k[0] + a * p.sC_k[ma],
                                        tile[0][tx][ty + 8 * r], CPLX ? tile[NC - 1][tx][ty + 8 * r] : 0.0);
    }
}

}  // namespace btc

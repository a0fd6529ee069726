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

// Nothing summed and dimension 0 contiguous in A, B and C alike: V consecutive elements (16 bytes)
// per thread, one vector load per input and one vector store.
template <typename R, bool CPLX, int V, typename I>
__global__ void __launch_bounds__(256) elementwise_vector_kernel(const ElementwiseParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    constexpr int W = V * NC;                            // words of type R per vector
    union Pack { uint4 raw; R w[W]; };
    static_assert(sizeof(R) * W == 16, "a vector is 16 bytes");
    const R *A = static_cast<const R *>(p.A);
    const R *B = static_cast<const R *>(p.B);
    R *C = static_cast<R *>(p.C);
    const int64_t nvec = p.total_keep / V;
    const int64_t stride = int64_t(gridDim.x) * blockDim.x;
    const R sgnA = (CPLX && p.conjA) ? R(-1) : R(1), sgnB = (CPLX && p.conjB) ? R(-1) : R(1);
    for (int64_t v = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; v < nvec; v += stride) {
        int64_t offA = 0, offB = 0, offC = 0;
        I lin = I(v);
        {
            const I ext = I(p.ext_k[0] / V);
            const I q = lin / ext;
            const int64_t i = int64_t(lin - q * ext) * V;
            lin = q;
            offA = i * p.sA_k[0]; offB = i * p.sB_k[0]; offC = i;
        }
        for (int d = 1; d < p.nk; ++d) {
            const I ext = I(p.ext_k[d]);
            const I q = lin / ext;
            const int64_t i = int64_t(lin - q * ext);
            lin = q;
            offA += i * p.sA_k[d];
            offB += i * p.sB_k[d];
            offC += i * p.sC_k[d];
        }
        Pack a, b, c;
        a.raw = make_uint4(0, 0, 0, 0);
        b.raw = make_uint4(0, 0, 0, 0);
        if (p.use_a) a.raw = *reinterpret_cast<const uint4 *>(A + NC * offA);
        if (p.use_b) b.raw = *reinterpret_cast<const uint4 *>(B + NC * offB);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            const double ar = p.use_a ? double(a.w[NC * e]) : 0.0;
            const double ai = (CPLX && p.use_a) ? double(sgnA * a.w[NC * e + (NC - 1)]) : 0.0;
            double c_r = p.alpha[0] * ar - p.alpha[1] * ai, c_i = p.alpha[0] * ai + p.alpha[1] * ar;
            if (p.use_b) {
                const double br = double(b.w[NC * e]);
                const double bi = CPLX ? double(sgnB * b.w[NC * e + (NC - 1)]) : 0.0;
                c_r += p.beta[0] * br - p.beta[1] * bi;
                c_i += p.beta[0] * bi + p.beta[1] * br;
            }
            c.w[NC * e] = R(c_r);
            if (CPLX) c.w[NC * e + (NC - 1)] = R(c_i);
        }
        *reinterpret_cast<uint4 *>(C + NC * offC) = c.raw;
    }
}

// blockIdx.x enumerates (tile along C's dimension 0, tile along A's dimension, rest), first fastest.
// T x T tiles (T = 64 for 4-byte elements, 32 otherwise: rows of at least 256 bytes on both sides),
// 256 threads, each T * T / 256 elements in either phase; the tile holds values already summed and
// rounded to the element type.
template <typename R, bool CPLX, typename I>
__global__ void __launch_bounds__(256) elementwise_transposing_kernel(const ElementwiseParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    constexpr int T = (sizeof(R) * NC == 4) ? 64 : 32;
    constexpr int ROWS = 256 / T;                        // tile rows covered by the CTA at once
    constexpr int PER = T / ROWS;                        // rows per thread
    __shared__ R tile[NC][T][T + 1];
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
    const int tx = threadIdx.x % T, ty = threadIdx.x / T;
    const int64_t c0 = tile_c * T, a0 = tile_a * T;
    const int64_t ext_c = p.ext_k[0], ext_a = p.ext_k[ma];
    // phase 1: consecutive threads along A's dimension
#pragma unroll
    for (int r = 0; r < PER; ++r) {
        const int64_t c = c0 + ty + ROWS * r, a = a0 + tx;
        double acc_r = 0.0, acc_i = 0.0;
        if (c < ext_c && a < ext_a)
            elementwise_sum<R, CPLX, 1, I>(p, restA + c * p.sA_k[0] + a * p.sA_k[ma], 0, acc_r, acc_i);
        tile[0][ty + ROWS * r][tx] = R(acc_r);
        if (CPLX) tile[NC - 1][ty + ROWS * r][tx] = R(acc_i);
    }
    __syncthreads();
    // phase 2: consecutive threads along C's dimension 0
#pragma unroll
    for (int r = 0; r < PER; ++r) {
        const int64_t c = c0 + tx, a = a0 + ty + ROWS * r;
        if (c < ext_c && a < ext_a)
            elementwise_finish<R, CPLX>(p, restB + c * p.sB_k[0] + a * p.sB_k[ma], restC + c * p.sC_k[0] + a * p.sC_k[ma],
                                        double(tile[0][tx][ty + ROWS * r]), CPLX ? double(tile[NC - 1][tx][ty + ROWS * r]) : 0.0);
    }
}

}  // namespace btc

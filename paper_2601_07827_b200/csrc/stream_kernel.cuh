// Bandwidth-bound contraction for very short contracted extents (K <= 4, in particular K = 1): outer
// products, Hadamard products, a scalar operand (permute-and-scale), rank-one updates -- the shapes of
// Appendix "Testing" items 1, 6 and 8 and Notes 2 and 4, for all four element types.  The result is
// as large as or far larger than the inputs, so the kernel is a streaming write of D: one thread per
// vector of V consecutive rows of D (V elements = 16 bytes where D is contiguous along its first M
// mode), enumerated with the row index fastest, then the column, then the batch entry, so that
// consecutive threads write consecutive vectors.  A thread reads its V elements of A and its one
// element of B per contracted index through the offset tables (neighbouring threads share them, so
// they come from L1 / L2), multiplies in the element type (double for the 64-bit types) and writes
// alpha * sum + beta * op(C) once.  Many small CTAs per SM keep enough loads and stores in flight; no
// shared memory, no barriers, nothing to wait for.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

constexpr int kStreamMaxK = 4;
constexpr int kStreamThreads = 256;

// complex multiply-add acc += op(a) * op(b); (ai, bi already negated by the caller when conjugated)
template <typename R>
__device__ __forceinline__ void cmac(R &cr, R &ci, R ar, R ai, R br, R bi)
{
    cr += ar * br - ai * bi;
    ci += ar * bi + ai * br;
}

// R: float / double; CPLX: interleaved (re, im); V: rows per thread: 1, or the number of elements in 16
// bytes, in which case the host guarantees that groups of V consecutive rows are V consecutive, 16-byte
// aligned elements of D (and C) and that M is a multiple of V; VEC_A: the same holds in A.
template <typename R, bool CPLX, int V, bool VEC_A>
__global__ void __launch_bounds__(kStreamThreads) stream_kernel(const TiledParams p)
{
    constexpr int W = CPLX ? 2 : 1;
    union Pack { uint4 raw; R w[V * W]; };                   // V elements; 16 bytes when V > 1
    const R *A = static_cast<const R *>(p.A), *B = static_cast<const R *>(p.B), *C = static_cast<const R *>(p.C);
    R *D = static_cast<R *>(p.D);
    const int64_t mv_count = (p.M + V - 1) / V;
    const int64_t total = mv_count * p.N * p.Bt;
    const int K = int(p.K);
    int64_t koA[kStreamMaxK], koB[kStreamMaxK];
#pragma unroll
    for (int k = 0; k < kStreamMaxK; ++k) {
        koA[k] = k < K ? p.offA_k[k] : 0;
        koB[k] = k < K ? p.offB_k[k] : 0;
    }
    const R sa = (CPLX && p.conjA) ? R(-1) : R(1), sb = (CPLX && p.conjB) ? R(-1) : R(1), sc = (CPLX && p.conjC) ? R(-1) : R(1);
    const R alr = R(p.alpha[0]), ali = R(p.alpha[1]), ber = R(p.beta[0]), bei = R(p.beta[1]);
    for (int64_t t = int64_t(blockIdx.x) * kStreamThreads + threadIdx.x; t < total; t += int64_t(gridDim.x) * kStreamThreads) {
        const int64_t mv = t % mv_count, rest = t / mv_count;
        const int64_t n = rest % p.N, h = rest / p.N;
        const int64_t m = mv * V;
        const int64_t oB = p.offB_n[n] + p.offB_h[h];
        const int64_t oD = p.offD_m[m] + p.offD_n[n] + p.offD_h[h];
        const int64_t oA = p.offA_m[m] + p.offA_h[h];
        R acc[V][W];
#pragma unroll
        for (int v = 0; v < V; ++v)
#pragma unroll
            for (int w = 0; w < W; ++w) acc[v][w] = R(0);
#pragma unroll
        for (int k = 0; k < kStreamMaxK; ++k) {
            if (k >= K) break;
            R b[W];
#pragma unroll
            for (int w = 0; w < W; ++w) b[w] = B[(oB + koB[k]) * W + w];
            if (CPLX) b[W - 1] *= sb;
            Pack a;
            if (V > 1 && VEC_A) {
                a.raw = *reinterpret_cast<const uint4 *>(A + (oA + koA[k]) * W);
            } else {
#pragma unroll
                for (int v = 0; v < V; ++v) {
                    const int64_t o = (v == 0 ? oA : p.offA_m[m + v] + p.offA_h[h]) + koA[k];
#pragma unroll
                    for (int w = 0; w < W; ++w) a.w[v * W + w] = A[o * W + w];
                }
            }
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (CPLX) cmac<R>(acc[v][0], acc[v][W - 1], a.w[v * W], sa * a.w[v * W + W - 1], b[0], b[W - 1]);
                else acc[v][0] += a.w[v] * b[0];
            }
        }
        // D = alpha * acc + beta * op(C)
        Pack c, d;
        if (p.use_c) {
            if (V > 1) c.raw = *reinterpret_cast<const uint4 *>(C + oD * W);
            else
#pragma unroll
                for (int w = 0; w < W; ++w) c.w[w] = C[oD * W + w];
        }
#pragma unroll
        for (int v = 0; v < V; ++v) {
            if (CPLX) {
                R dr = alr * acc[v][0] - ali * acc[v][W - 1], di = alr * acc[v][W - 1] + ali * acc[v][0];
                if (p.use_c) {
                    const R cr = c.w[v * W], ci = sc * c.w[v * W + W - 1];
                    dr += ber * cr - bei * ci;
                    di += ber * ci + bei * cr;
                }
                d.w[v * W] = dr;
                d.w[v * W + W - 1] = di;
            } else {
                R dr = alr * acc[v][0];
                if (p.use_c) dr += ber * c.w[v];
                d.w[v] = dr;
            }
        }
        if (V > 1) *reinterpret_cast<uint4 *>(D + oD * W) = d.raw;
        else
#pragma unroll
            for (int w = 0; w < W; ++w) D[oD * W + w] = d.w[w];
    }
}

}  // namespace btc

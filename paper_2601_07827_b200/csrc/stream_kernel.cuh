// Bandwidth-bound contraction for very short contracted extents (K <= 4, in particular K = 1): outer
// products, Hadamard products, a scalar operand (permute-and-scale), rank-one updates -- the shapes of
// Appendix "Testing" items 1, 6 and 8 and Notes 2 and 4, for all four element types.  The result is
// as large as or far larger than the inputs, so the kernel is a streaming write of D: a thread owns a
// vector of V consecutive rows of D (V elements = 16 bytes where D is contiguous along its first M
// mode) of one batch entry, keeps the matching elements of A in registers and walks a few columns,
// reading one element of B per column and contracted index (shared by the CTA, so it comes from L1)
// and writing alpha * sum + beta * op(C) with one 16-byte store per column; consecutive threads own
// consecutive row vectors, so a warp's store is one run of 512 bytes where D is contiguous that far.
// Products and sums are formed in the element type (double for the 64-bit types).  Many small CTAs per
// SM keep enough loads and stores in flight; no shared memory, no barriers, nothing to wait for.
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

constexpr int kStreamColumns = 32;       // columns of D a thread walks with one row vector in registers

// R: float / double; CPLX: interleaved (re, im); V: rows per thread: 1, or the number of elements in 16
// bytes, in which case the host guarantees that groups of V consecutive rows are V consecutive, 16-byte
// aligned elements of D (and C) and that M is a multiple of V; VEC_A: the same holds in A.
// Work split: x = (row vector, batch entry), row vector fastest; y = column.  A CTA covers txv consecutive x
// (a power of two <= 256, chosen by the host so that short x ranges leave threads for the columns) times
// (256 / txv) * kStreamColumns consecutive y; a thread keeps its x -- offsets and, per contracted index,
// its V elements of A -- in registers and walks its columns, so the integer divisions and the row-side
// table look-ups are paid once per thread, not once per element.
template <typename R, bool CPLX, int V, bool VEC_A>
__global__ void __launch_bounds__(kStreamThreads) stream_kernel(const TiledParams p, int txv, int64_t x_blocks)
{
    constexpr int W = CPLX ? 2 : 1;
    union Pack { uint4 raw; R w[V * W]; };                   // V elements; 16 bytes when V > 1
    const R *A = static_cast<const R *>(p.A), *B = static_cast<const R *>(p.B), *C = static_cast<const R *>(p.C);
    R *D = static_cast<R *>(p.D);
    const int64_t mv_count = (p.M + V - 1) / V, x_count = mv_count * p.Bt;
    const int K = int(p.K);
    const int tyt = kStreamThreads / txv;                    // threads along y
    const int64_t bx = int64_t(blockIdx.x) % x_blocks, by = int64_t(blockIdx.x) / x_blocks;
    const int64_t x = bx * txv + int(threadIdx.x) % txv;
    const int64_t y0 = by * (int64_t(tyt) * kStreamColumns) + int(threadIdx.x) / txv;
    if (x >= x_count) return;
    const int64_t m = (x % mv_count) * V, h = x / mv_count;
    const int64_t hB = p.offB_h[h];
    const int64_t xD = p.offD_m[m] + p.offD_h[h];
    const int64_t xA = p.offA_m[m] + p.offA_h[h];
    const R sa = (CPLX && p.conjA) ? R(-1) : R(1), sb = (CPLX && p.conjB) ? R(-1) : R(1), sc = (CPLX && p.conjC) ? R(-1) : R(1);
    const R alr = R(p.alpha[0]), ali = R(p.alpha[1]), ber = R(p.beta[0]), bei = R(p.beta[1]);
    // this thread's rows of A, one vector per contracted index (imaginary parts already conjugated)
    Pack a[kStreamMaxK];
    int64_t koB[kStreamMaxK];
#pragma unroll
    for (int k = 0; k < kStreamMaxK; ++k) {
        koB[k] = 0;
        if (k >= K) continue;
        koB[k] = p.offB_k[k] + hB;
        const int64_t ko = p.offA_k[k];
#ifdef BTC_CHECK_OFFSETS
        for (int v = 0; v < V; ++v)
            if (!BTC_IN_SPAN(p.spans, 0, ((V > 1 && VEC_A) ? xA + v : p.offA_m[m + v] + p.offA_h[h]) + ko, 1)) return;
#endif
        if (V > 1 && VEC_A) {
            a[k].raw = *reinterpret_cast<const uint4 *>(A + (xA + ko) * W);
        } else {
#pragma unroll
            for (int v = 0; v < V; ++v) {
                const int64_t o = (v == 0 ? xA : p.offA_m[m + v] + p.offA_h[h]) + ko;
#pragma unroll
                for (int w = 0; w < W; ++w) a[k].w[v * W + w] = A[o * W + w];
            }
        }
        if (CPLX)
#pragma unroll
            for (int v = 0; v < V; ++v) a[k].w[v * W + W - 1] *= sa;
    }
#pragma unroll 2
    for (int j = 0; j < kStreamColumns; ++j) {
        const int64_t y = y0 + int64_t(j) * tyt;
        if (y >= p.N) break;
        const int64_t oB = p.offB_n[y];
        const int64_t oD = xD + p.offD_n[y];
#ifdef BTC_CHECK_OFFSETS
        bool in_span = BTC_IN_SPAN(p.spans, 2, oD, V);
        for (int k = 0; k < K; ++k) in_span = in_span && BTC_IN_SPAN(p.spans, 1, oB + koB[k], 1);
        if (!in_span) continue;
#endif
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
#pragma unroll
            for (int v = 0; v < V; ++v) {
                if (CPLX) cmac<R>(acc[v][0], acc[v][W - 1], a[k].w[v * W], a[k].w[v * W + W - 1], b[0], b[W - 1]);
                else acc[v][0] += a[k].w[v] * b[0];
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

// C := alpha op(A) + beta op(B)  (Sec. "Unary and Binary Operations"): labels only in A are summed
// over, A is broadcast along labels only in C, repeated labels of A act through summed strides.
// All kernels are bandwidth-bound passes: A (and B) read once through their strides, C written
// once through its own.
//   direct       one thread (or one warp, lanes over the summed index) per element of C, C's
//                most contiguous dimension fastest.  Right when A is contiguous along the same
//                dimension (scaling, addition, reduction, broadcast).
//   transposing  permutations whose input is contiguous along another dimension than the output:
//                a CTA moves a tile (128 x 64 elements of 4 bytes, 64 x 64 of 8, 32 x 32 of 16) through
//                shared memory, reading along A's dimension and writing along C's, so both sides
//                move rows of 256-512 bytes.
//   vector       nothing summed and dimension 0 contiguous in every tensor: 16-byte vectors.
// Sums are kept in double (pairs for complex) for every element type.
#pragma once

#include <cuda_runtime.h>

#include "isolated_sum_kernel.cuh"
#include "kernel_params.h"

namespace btc {

// lin / ext for the loop dimension `d` of p (kGenericMaxD: dimension 0 counted in vectors): 32-bit indices
// multiply by the reciprocal prepared on the host, 64-bit indices divide
template <typename I>
__device__ __forceinline__ I elementwise_div(const ElementwiseParams &p, I lin, I ext, int d)
{
    if (sizeof(I) == 4) return I((uint64_t(uint32_t(lin)) * p.div_mul[d]) >> p.div_shift[d]);
    return lin / ext;
}

// arithmetic type of alpha * a + beta * b where nothing is summed: the part type itself
template <typename R> struct ElementwiseScalar { typedef R type; };

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
    constexpr int U = LANES == 1 ? 8 : 4;   // loads in flight per thread (16 spill: 4x slower)
    const R *A = static_cast<const R *>(p.A);
    acc_r = acc_i = 0.0;
    if (!p.use_a) return;
    if (p.ns == 0) {                       // nothing to sum: one element
        if (lane == 0) {
            acc_r = double(A[NC * base]);
            if (CPLX) acc_i = double(A[NC * base + (NC - 1)]);
        }
    } else if (p.ns == 1) {
        // one summed dimension: a running pointer, whole groups of U loads without bounds tests
        const int64_t step = NC * LANES * p.sA_s[0];
        const R *q = A + NC * (base + lane * p.sA_s[0]);
        int64_t left = (p.total_sum - lane + LANES - 1) / LANES;      // this lane's share of the summed index
        if (left < 0) left = 0;
        for (; left >= U; left -= U) {
            R v_r[U], v_i[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                v_r[u] = q[u * step];
                v_i[u] = CPLX ? q[u * step + (NC - 1)] : R(0);
            }
            q += U * step;
#pragma unroll
            for (int u = 0; u < U; ++u) {
                acc_r += double(v_r[u]);
                if (CPLX) acc_i += double(v_i[u]);
            }
        }
        for (; left > 0; --left) {
            acc_r += double(q[0]);
            if (CPLX) acc_i += double(q[NC - 1]);
            q += step;
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
    if (LANES == 1 && p.ns == 0) {
        // nothing summed: four elements per thread and pass, all loads issued before the first
        // store (B may be C's memory, so the compiler would not move them by itself)
        constexpr int NC = CPLX ? 2 : 1;
        constexpr int U = 4;
        const R *A = static_cast<const R *>(p.A);
        const R *B = static_cast<const R *>(p.B);
        R *C = static_cast<R *>(p.C);
        for (int64_t e0 = group; e0 < p.total_keep; e0 += int64_t(U) * ngroups) {
            int64_t offA[U], offB[U], offC[U];
            bool in[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t e = e0 + int64_t(u) * ngroups;
                in[u] = e < p.total_keep;
                offA[u] = offB[u] = offC[u] = 0;
                I lin = I(in[u] ? e : 0);
                for (int d = 0; d < p.nk; ++d) {
                    const I ext = I(p.ext_k[d]);
                    const I q = elementwise_div<I>(p, lin, ext, d);
                    const int64_t i = int64_t(lin - q * ext);
                    lin = q;
                    offA[u] += i * p.sA_k[d];
                    offB[u] += i * p.sB_k[d];
                    offC[u] += i * p.sC_k[d];
                }
            }
            R a_r[U], a_i[U], b_r[U], b_i[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                a_r[u] = (p.use_a && in[u]) ? A[NC * offA[u]] : R(0);
                a_i[u] = (CPLX && p.use_a && in[u]) ? A[NC * offA[u] + (NC - 1)] : R(0);
                b_r[u] = (p.use_b && in[u]) ? B[NC * offB[u]] : R(0);
                b_i[u] = (CPLX && p.use_b && in[u]) ? B[NC * offB[u] + (NC - 1)] : R(0);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (!in[u]) continue;
                typedef typename ElementwiseScalar<R>::type S;
                const S al_r = S(p.alpha[0]), al_i = S(p.alpha[1]), be_r = S(p.beta[0]), be_i = S(p.beta[1]);
                const S ar = S(a_r[u]), ai = p.conjA ? -S(a_i[u]) : S(a_i[u]);
                const S br = S(b_r[u]), bi = p.conjB ? -S(b_i[u]) : S(b_i[u]);
                if (CPLX) {
                    C[NC * offC[u]] = R(al_r * ar - al_i * ai + be_r * br - be_i * bi);
                    C[NC * offC[u] + (NC - 1)] = R(al_r * ai + al_i * ar + be_r * bi + be_i * br);
                } else {
                    C[NC * offC[u]] = R(al_r * ar + be_r * br);
                }
            }
        }
        return;
    }
    for (int64_t e = group; e < p.total_keep; e += ngroups) {
        int64_t offA = 0, offB = 0, offC = 0;
        I lin = I(e);
        for (int d = 0; d < p.nk; ++d) {
            const I ext = I(p.ext_k[d]);
            const I q = elementwise_div<I>(p, lin, ext, d);
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
    typedef typename ElementwiseScalar<R>::type S;
    const S al_r = S(p.alpha[0]), al_i = S(p.alpha[1]), be_r = S(p.beta[0]), be_i = S(p.beta[1]);
    constexpr int U = 4;                                 // vectors in flight per thread
    for (int64_t v0 = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; v0 < nvec; v0 += int64_t(U) * stride) {
        int64_t offA[U], offB[U], offC[U];
        bool in[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int64_t v = v0 + int64_t(u) * stride;
            in[u] = v < nvec;
            I lin = I(in[u] ? v : 0);
            const I ext0 = I(p.ext_k[0] / V);
            const I q0 = elementwise_div<I>(p, lin, ext0, kGenericMaxD);
            const int64_t i0 = int64_t(lin - q0 * ext0) * V;
            lin = q0;
            offA[u] = i0 * p.sA_k[0]; offB[u] = i0 * p.sB_k[0]; offC[u] = i0;
            for (int d = 1; d < p.nk; ++d) {
                const I ext = I(p.ext_k[d]);
                const I q = elementwise_div<I>(p, lin, ext, d);
                const int64_t i = int64_t(lin - q * ext);
                lin = q;
                offA[u] += i * p.sA_k[d];
                offB[u] += i * p.sB_k[d];
                offC[u] += i * p.sC_k[d];
            }
        }
        Pack a[U], b[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            a[u].raw = make_uint4(0, 0, 0, 0);
            b[u].raw = make_uint4(0, 0, 0, 0);
            if (p.use_a && in[u]) a[u].raw = *reinterpret_cast<const uint4 *>(A + NC * offA[u]);
            if (p.use_b && in[u]) b[u].raw = *reinterpret_cast<const uint4 *>(B + NC * offB[u]);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (!in[u]) continue;
            Pack c;
#pragma unroll
            for (int e = 0; e < V; ++e) {
                const S ar = S(a[u].w[NC * e]), br = S(b[u].w[NC * e]);
                if (CPLX) {
                    const S ai = S(sgnA * a[u].w[NC * e + (NC - 1)]), bi = S(sgnB * b[u].w[NC * e + (NC - 1)]);
                    c.w[NC * e] = R(al_r * ar - al_i * ai + be_r * br - be_i * bi);
                    c.w[NC * e + (NC - 1)] = R(al_r * ai + al_i * ar + be_r * bi + be_i * br);
                } else {
                    c.w[NC * e] = R(al_r * ar + be_r * br);
                }
            }
            *reinterpret_cast<uint4 *>(C + NC * offC[u]) = c.raw;
        }
    }
}

// Tile and CTA size of the transposing kernel, 256 threads: 128 (along C's dimension 0) x 64 (along A's
// dimension) for 4-byte elements, 64 x 64 for 8-byte ones, 32 x 32 for complex128, i.e. rows of 512 bytes
// where shared memory and registers allow.  Measured on permutations of 1 GB fp32 tensors: 64 x 64
// (256-byte rows) 5.0-5.4 TB/s, 128 x 64 or 64 x 128 6.0-6.3 TB/s, 128 x 128 with 1024 threads 3.6 TB/s
// (two large CTAs per SM overlap poorly).
template <typename R, bool CPLX> struct TransposeTile {
    static constexpr int NC = CPLX ? 2 : 1;
    static constexpr int T = sizeof(R) * NC <= 8 ? 64 : 32;
    // tile extent along C's dimension 0 (rows written) and along A's dimension (rows read)
    static constexpr int TC = sizeof(R) * NC == 4 ? 128 : T, TA = T;
    static constexpr int THREADS = 256;
    static constexpr size_t SMEM_BYTES = size_t(NC) * TC * (TA + 1) * sizeof(R);
};

// blockIdx.x enumerates (tile along C's dimension 0, tile along A's dimension, rest), first fastest.
// Each thread handles TC * TA / THREADS elements in either phase; the tile holds values already
// summed and rounded to the element type.
// SUMS: compiled with the branches for summed dimensions (and for alpha = 0); the pure permutation
// is a kernel of its own, so that it keeps its register count and occupancy.
template <typename R, bool CPLX, typename I, bool SUMS>
__global__ void __launch_bounds__((TransposeTile<R, CPLX>::THREADS)) elementwise_transposing_kernel(const ElementwiseParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    constexpr int TC = TransposeTile<R, CPLX>::TC, TA = TransposeTile<R, CPLX>::TA;
    constexpr int ROWS1 = TransposeTile<R, CPLX>::THREADS / TA, PER1 = TC / ROWS1;   // phase 1: rows of TA along A's dimension
    constexpr int ROWS2 = TransposeTile<R, CPLX>::THREADS / TC, PER2 = TA / ROWS2;   // phase 2: rows of TC along C's dimension 0
    extern __shared__ __align__(16) unsigned char tile_bytes[];
    R (*tile)[TC][TA + 1] = reinterpret_cast<R (*)[TC][TA + 1]>(tile_bytes);
    const int ma = p.tile_mode_a;
    // (32-bit arithmetic: the grid has fewer than 2^31 CTAs; an extent of 2^31 or more has no
    // reciprocal -- its multiplier is 0 -- and the quotient 0 that comes out is the right one)
    const uint32_t q_c = blockIdx.x / uint32_t(p.tiles_c), q_a = q_c / uint32_t(p.tiles_a);
    const int64_t tile_c = blockIdx.x - q_c * uint32_t(p.tiles_c);
    const int64_t tile_a = q_c - q_a * uint32_t(p.tiles_a);
    uint32_t lin = q_a;
    int64_t restA = 0, restB = 0, restC = 0;
    for (int d = 1; d < p.nk; ++d) {
        if (d == ma) continue;
        const uint32_t q = elementwise_div<uint32_t>(p, lin, uint32_t(p.ext_k[d]), d);
        const int64_t i = int64_t(lin - q * uint32_t(p.ext_k[d]));
        lin = q;
        restA += i * p.sA_k[d];
        restB += i * p.sB_k[d];
        restC += i * p.sC_k[d];
    }
    const int64_t c0 = tile_c * TC, a0 = tile_a * TA;
    const int64_t ext_c = p.ext_k[0], ext_a = p.ext_k[ma];
    // phase 1: consecutive threads along A's dimension.  Without summed dimensions (a pure
    // permutation) all of a thread's loads are issued before the first value is used; a load
    // inside the bounds test of its own iteration would leave one load in flight per thread.
    {
    const int tx = threadIdx.x % TA, ty = threadIdx.x / TA;
    if (!SUMS) {
        const R *A = static_cast<const R *>(p.A);
        R v_r[PER1], v_i[PER1];
        const bool a_in = a0 + tx < ext_a;
        const R *src = A + NC * (restA + (a0 + tx) * p.sA_k[ma] + (c0 + ty) * p.sA_k[0]);
        const int64_t step = NC * ROWS1 * p.sA_k[0];
        const int rows_in = int(ext_c - c0 - ty < int64_t(TC) ? ext_c - c0 - ty : int64_t(TC));   // rows ty + ROWS1 r < rows_in exist
#pragma unroll
        for (int r = 0; r < PER1; ++r) {
            const bool in = a_in && ROWS1 * r < rows_in;
            v_r[r] = in ? src[0] : R(0);
            v_i[r] = (CPLX && in) ? src[NC - 1] : R(0);
            src += step;
        }
#pragma unroll
        for (int r = 0; r < PER1; ++r) {
            tile[0][ty + ROWS1 * r][tx] = v_r[r];
            if (CPLX) tile[NC - 1][ty + ROWS1 * r][tx] = p.conjA ? -v_i[r] : v_i[r];
        }
    } else if (SUMS && p.ns == 1 && p.use_a) {
        // One summed dimension (the usual case after chained dimensions are merged): a running pointer per
        // row instead of an index decode per element, eight loads in flight, whole groups of eight without
        // bounds tests (an element costs a load, a conversion and an add: the loop is issue-bound otherwise).
        const R *A = static_cast<const R *>(p.A);
        const int64_t step = NC * p.sA_s[0];
        const bool a_in = a0 + tx < ext_a;
        const R *row0 = A + NC * (restA + (a0 + tx) * p.sA_k[ma] + (c0 + ty) * p.sA_k[0]);
        const int64_t rstep = NC * ROWS1 * p.sA_k[0];
        const int rows_in = int(ext_c - c0 - ty < int64_t(TC) ? ext_c - c0 - ty : int64_t(TC));   // rows ty + ROWS1 r < rows_in exist
#pragma unroll 1
        for (int r = 0; r < PER1; ++r) {
            double acc_r = 0.0, acc_i = 0.0;
            if (a_in && ROWS1 * r < rows_in) {
                const R *q = row0 + r * rstep;
                int64_t left = p.total_sum;
                for (; left >= 8; left -= 8) {
                    R v_r[8], v_i[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        v_r[u] = q[u * step];
                        v_i[u] = CPLX ? q[u * step + (NC - 1)] : R(0);
                    }
                    q += 8 * step;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        acc_r += double(v_r[u]);
                        if (CPLX) acc_i += double(v_i[u]);
                    }
                }
                for (; left > 0; --left) {
                    acc_r += double(q[0]);
                    if (CPLX) acc_i += double(q[NC - 1]);
                    q += step;
                }
            }
            tile[0][ty + ROWS1 * r][tx] = R(acc_r);
            if (CPLX) tile[NC - 1][ty + ROWS1 * r][tx] = R(p.conjA ? -acc_i : acc_i);   // conjugation commutes with the sum
        }
    } else {
#pragma unroll
        for (int r = 0; r < PER1; ++r) {
            const int64_t c = c0 + ty + ROWS1 * r, a = a0 + tx;
            double acc_r = 0.0, acc_i = 0.0;
            if (c < ext_c && a < ext_a)
                elementwise_sum<R, CPLX, 1, I>(p, restA + c * p.sA_k[0] + a * p.sA_k[ma], 0, acc_r, acc_i);
            tile[0][ty + ROWS1 * r][tx] = R(acc_r);
            if (CPLX) tile[NC - 1][ty + ROWS1 * r][tx] = R(acc_i);
        }
    }
    }
    __syncthreads();
    // phase 2: consecutive threads along C's dimension 0; B's values are loaded as a batch too
    // (B may be the same memory as C, so the compiler cannot move its loads across the stores).
    // alpha * t + beta * b is formed in double only for 64-bit parts: for 32-bit parts the two
    // products and the sum in float are within a few units in the last place of |alpha t| + |beta b|.
    {
        const int tx = threadIdx.x % TC, ty = threadIdx.x / TC;
        typedef typename ElementwiseScalar<R>::type S;
        const R *B = static_cast<const R *>(p.B);
        R *C = static_cast<R *>(p.C);
        const bool c_in = c0 + tx < ext_c;
        const int rows_in = int(ext_a - a0 - ty < int64_t(TA) ? ext_a - a0 - ty : int64_t(TA));
        const R *srcB = B + NC * (restB + (c0 + tx) * p.sB_k[0] + (a0 + ty) * p.sB_k[ma]);
        R *dst = C + NC * (restC + (c0 + tx) * p.sC_k[0] + (a0 + ty) * p.sC_k[ma]);
        const int64_t stepB = NC * ROWS2 * p.sB_k[ma], stepC = NC * ROWS2 * p.sC_k[ma];
        const S al_r = S(p.alpha[0]), al_i = S(p.alpha[1]), be_r = S(p.beta[0]), be_i = S(p.beta[1]);
        R b_r[PER2], b_i[PER2];
#pragma unroll
        for (int r = 0; r < PER2; ++r) {
            const bool in = p.use_b && c_in && ROWS2 * r < rows_in;
            b_r[r] = in ? srcB[0] : R(0);
            b_i[r] = (CPLX && in) ? srcB[NC - 1] : R(0);
            srcB += stepB;
        }
#pragma unroll
        for (int r = 0; r < PER2; ++r) {
            if (c_in && ROWS2 * r < rows_in) {
                const S t_r = S(tile[0][tx][ty + ROWS2 * r]), t_i = CPLX ? S(tile[NC - 1][tx][ty + ROWS2 * r]) : S(0);
                const S br = S(b_r[r]), bi = CPLX ? (p.conjB ? -S(b_i[r]) : S(b_i[r])) : S(0);
                if (CPLX) {
                    dst[0] = R(al_r * t_r - al_i * t_i + be_r * br - be_i * bi);
                    dst[NC - 1] = R(al_r * t_i + al_i * t_r + be_r * bi + be_i * br);
                } else {
                    dst[0] = R(al_r * t_r + be_r * br);
                }
            }
            dst += stepC;
        }
    }
}

}  // namespace btc

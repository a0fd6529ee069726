// Case 4 of Sec. "Operations": a label that occurs in only one input tensor is summed over before
// the contraction,  X'[kept] = sum over the isolated labels of X[kept, isolated].
// A bandwidth-bound pass: X is read once through its strides, X' is written densely (kept labels
// in order of increasing |stride| in X, so consecutive threads read and write neighbouring
// elements).  LANES = 1: one thread per element of X'.  LANES = 32: one warp per element, lanes
// striding over the isolated index, for tensors whose isolated label is the contiguous one; where that
// label's runs are whole 16-byte vectors, the vector kernel at the end of this file runs instead.
// Sums are kept in double (pairs for complex) for every element type; conjugation commutes with
// the sum and stays with the contraction.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

// Mixed-radix decode of a linear index into an element offset; 32-bit arithmetic when it fits
// (64-bit division costs an order of magnitude more instructions).
template <typename I>
__device__ __forceinline__ int64_t decode_offset(I lin, int nd, const int64_t *ext, const int64_t *str)
{
    if (nd == 1) return int64_t(lin) * str[0];      // the common case after chained dimensions are merged
    int64_t off = 0;
    for (int d = 0; d < nd; ++d) {
        const I e = I(ext[d]);
        const I q = lin / e;
        off += int64_t(lin - q * e) * str[d];
        lin = q;
    }
    return off;
}

template <typename R, bool CPLX, int LANES, typename I>
__global__ void __launch_bounds__(256) isolated_sum_kernel(const IsolatedSumParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    // independent loads in flight per thread: LANES = 1 unrolls the isolated index of one result
    // element, LANES = 32 works on several result elements at a time
    constexpr int U = LANES == 1 ? 8 : 1, E = LANES == 1 ? 1 : 4;
    const R *src = static_cast<const R *>(p.src);
    R *dst = static_cast<R *>(p.dst);
    const int lane = (LANES == 1) ? 0 : int(threadIdx.x) % LANES;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) / LANES;
    const int64_t ngroups = (int64_t(gridDim.x) * blockDim.x) / LANES;
    for (int64_t e0 = group; e0 < p.total_keep; e0 += ngroups * E) {
        int64_t base[E];
        bool live[E];
        double acc_r[E], acc_i[E];
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const int64_t e = e0 + j * ngroups;
            live[j] = e < p.total_keep;
            base[j] = live[j] ? decode_offset<I>(I(e), p.nk, p.ext_k, p.str_k) : 0;
            acc_r[j] = acc_i[j] = 0.0;
        }
        if (LANES == 1 && p.ni == 1) {
            // one isolated dimension, one result element per thread: a running pointer and whole groups of
            // eight loads without bounds tests (the general loop below is bound by instruction issue for
            // 4-byte elements: an index decode and a test per load)
            if (live[0]) {
                const int64_t step = NC * p.str_i[0];
                const R *q = src + NC * base[0];
                int64_t left = p.total_iso;
                for (; left >= 8; left -= 8) {
                    R w_r[8], w_i[8];
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        w_r[u] = q[u * step];
                        w_i[u] = CPLX ? q[u * step + (NC - 1)] : R(0);
                    }
                    q += 8 * step;
#pragma unroll
                    for (int u = 0; u < 8; ++u) {
                        acc_r[0] += double(w_r[u]);
                        if (CPLX) acc_i[0] += double(w_i[u]);
                    }
                }
                for (; left > 0; --left) {
                    acc_r[0] += double(q[0]);
                    if (CPLX) acc_i[0] += double(q[NC - 1]);
                    q += step;
                }
            }
        } else
        for (int64_t s0 = lane; s0 < p.total_iso; s0 += int64_t(U) * LANES) {
            R v_r[E][U], v_i[E][U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int64_t s = s0 + int64_t(u) * LANES;
                const bool in_s = s < p.total_iso;
                const int64_t so = in_s ? decode_offset<I>(I(s), p.ni, p.ext_i, p.str_i) : 0;
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    const bool in = in_s && live[j];
                    v_r[j][u] = in ? src[NC * (base[j] + so)] : R(0);
                    v_i[j][u] = (CPLX && in) ? src[NC * (base[j] + so) + (NC - 1)] : R(0);
                }
            }
#pragma unroll
            for (int j = 0; j < E; ++j)
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    acc_r[j] += double(v_r[j][u]);
                    if (CPLX) acc_i[j] += double(v_i[j][u]);
                }
        }
#pragma unroll
        for (int j = 0; j < E; ++j) {
            if (LANES > 1) {
#pragma unroll
                for (int o = LANES / 2; o > 0; o >>= 1) {
                    acc_r[j] += __shfl_xor_sync(0xffffffffu, acc_r[j], o);
                    if (CPLX) acc_i[j] += __shfl_xor_sync(0xffffffffu, acc_i[j], o);
                }
            }
            const int64_t e = e0 + j * ngroups;
            if (lane == 0 && e < p.total_keep) {
                dst[NC * e] = R(acc_r[j]);
                if (CPLX) dst[NC * e + (NC - 1)] = R(acc_i[j]);
            }
        }
    }
}

// The isolated index is the contiguous one (stride 1, a multiple of 16 bytes long, every kept stride a
// multiple of 16 bytes too): L = 2^LOG_L neighbouring lanes share a result element, each lane reads
// 16-byte vectors L vectors apart (the L lanes together one run of 16 L bytes), sums its own vectors
// in registers and the lanes finish with LOG_L shuffle steps.  E = 2 result elements per lane group are in
// flight at a time (measured: 4 or 8 are slower, the reads then come from more places at once).
template <typename R, bool CPLX, int LOG_L, typename I>
__global__ void __launch_bounds__(256) isolated_sum_vector_kernel(const IsolatedSumParams p)
{
    constexpr int NC = CPLX ? 2 : 1, L = 1 << LOG_L;
    constexpr int W = 16 / int(sizeof(R));             // words of type R per vector
    constexpr int V = W / NC;                          // elements per vector
    constexpr int E = 2, U = 2;
    union Pack { uint4 raw; R w[W]; };
    const R *src = static_cast<const R *>(p.src);
    R *dst = static_cast<R *>(p.dst);
    const int sub = int(threadIdx.x) & (L - 1);
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) >> LOG_L;
    const int64_t ngroups = (int64_t(gridDim.x) * blockDim.x) >> LOG_L;
    const int64_t nvec = p.total_iso / V;
    // every lane of a warp runs the same number of passes (the shuffles below need all of them)
    const int64_t group_w = (int64_t(blockIdx.x) * blockDim.x + (threadIdx.x & ~31u)) >> LOG_L;      // the warp's first group
    for (int64_t pass = 0; group_w + pass < p.total_keep; pass += ngroups * E) {
        const int64_t e0 = group + pass;
        int64_t base[E];
        bool live[E];
        double acc_r[E], acc_i[E];
#pragma unroll
        for (int j = 0; j < E; ++j) {
            const int64_t e = e0 + j * ngroups;
            live[j] = e < p.total_keep;
            base[j] = live[j] ? decode_offset<I>(I(e), p.nk, p.ext_k, p.str_k) : 0;
            acc_r[j] = acc_i[j] = 0.0;
        }
        for (int64_t v0 = sub; v0 < nvec; v0 += int64_t(U) * L) {
            Pack x[E][U];
#pragma unroll
            for (int u = 0; u < U; ++u)
#pragma unroll
                for (int j = 0; j < E; ++j) {
                    const int64_t v = v0 + int64_t(u) * L;
                    x[j][u].raw = make_uint4(0, 0, 0, 0);
                    if (live[j] && v < nvec) x[j][u].raw = *reinterpret_cast<const uint4 *>(src + NC * (base[j] + v * V));
                }
#pragma unroll
            for (int j = 0; j < E; ++j)
#pragma unroll
                for (int u = 0; u < U; ++u)
#pragma unroll
                    for (int w = 0; w < W; ++w) {
                        if (CPLX && (w & 1)) acc_i[j] += double(x[j][u].w[w]);
                        else acc_r[j] += double(x[j][u].w[w]);
                    }
        }
#pragma unroll
        for (int j = 0; j < E; ++j) {
#pragma unroll
            for (int o = L / 2; o > 0; o >>= 1) {
                acc_r[j] += __shfl_xor_sync(0xffffffffu, acc_r[j], o);
                if (CPLX) acc_i[j] += __shfl_xor_sync(0xffffffffu, acc_i[j], o);
            }
            const int64_t e = e0 + j * ngroups;
            if (sub == 0 && e < p.total_keep) {
                dst[NC * e] = R(acc_r[j]);
                if (CPLX) dst[NC * e + (NC - 1)] = R(acc_i[j]);
            }
        }
    }
}

}  // namespace btc

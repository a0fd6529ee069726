// Case 4 of Sec. "Operations": a label that occurs in only one input tensor is summed over before
// the contraction,  X'[kept] = sum over the isolated labels of X[kept, isolated].
// A bandwidth-bound pass: X is read once through its strides, X' is written densely (kept labels
// in order of increasing |stride| in X, so consecutive threads read and write neighbouring
// elements).  LANES = 1: one thread per element of X'.  LANES = 32: one warp per element, lanes
// striding over the isolated index, for tensors whose isolated label is the contiguous one.
// Sums are kept in double (pairs for complex) for every element type; conjugation commutes with
// the sum and stays with the contraction.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

template <typename R, bool CPLX, int LANES>
__global__ void __launch_bounds__(256) isolated_sum_kernel(const IsolatedSumParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    const R *src = static_cast<const R *>(p.src);
    R *dst = static_cast<R *>(p.dst);
    const int lane = (LANES == 1) ? 0 : int(threadIdx.x) % LANES;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) / LANES;
    const int64_t ngroups = (int64_t(gridDim.x) * blockDim.x) / LANES;
    for (int64_t e = group; e < p.total_keep; e += ngroups) {
        int64_t base = 0, lin = e;
        for (int d = 0; d < p.nk; ++d) {
            base += (lin % p.ext_k[d]) * p.str_k[d];
            lin /= p.ext_k[d];
        }
        double acc_r = 0.0, acc_i = 0.0;
        for (int64_t s = lane; s < p.total_iso; s += LANES) {
            int64_t off = base, r = s;
            for (int d = 0; d < p.ni; ++d) {
                off += (r % p.ext_i[d]) * p.str_i[d];
                r /= p.ext_i[d];
            }
            acc_r += double(src[NC * off]);
            if (CPLX) acc_i += double(src[NC * off + (NC - 1)]);
        }
        if (LANES > 1) {
#pragma unroll
            for (int o = LANES / 2; o > 0; o >>= 1) {
                acc_r += __shfl_xor_sync(0xffffffffu, acc_r, o);
                if (CPLX) acc_i += __shfl_xor_sync(0xffffffffu, acc_i, o);
            }
        }
        if (lane == 0) {
            dst[NC * e] = R(acc_r);
            if (CPLX) dst[NC * e + (NC - 1)] = R(acc_i);
        }
    }
}

}  // namespace btc

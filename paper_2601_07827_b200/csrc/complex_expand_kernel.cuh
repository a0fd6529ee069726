// complex64 contractions on the fp32 tensor-core path: the real form of a complex product.
//
// D = alpha op(X) op(Y) over complex numbers is a real contraction once X is replaced by the 2 x 2
// real matrices of its elements: with x~ = alpha op(x), y = (yr, yi) and s = -1 where Y is conjugated,
//     Dr = x~r yr - s x~i yi,      Di = x~i yr + s x~r yi,
// so  D'[v, ...] = sum over u of X''[v, u, ...] Y'[u, ...]   with  X''[0][0] = x~r, X''[0][1] = -s x~i,
//                                                                  X''[1][0] = x~i, X''[1][1] =  s x~r,
// where Y' and D' are Y and D read as real tensors with one more mode (u, v: real / imaginary part,
// stride 1) and u is one more contracted label.  The host picks the smaller input as X, this kernel
// writes X'' (dense, in the caller's workspace) and the fp32 kernels run the real contraction (Eq. (case2)
// holds for it unchanged); conjugation of both inputs and alpha live in X''.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

namespace btc {

constexpr int kExpandMaxD = 32;

// Loop dimensions of X in the order of X'' (contracted ones first, `nkc` of them with `total_k`
// elements together, then the others): extent and stride in X (complex elements).  X'' holds, for the
// element with linear index lin_k + total_k * lin_rest, the four floats at 2 lin_k + 4 total_k lin_rest
// + u + 2 total_k v.
struct ComplexExpandParams {
    const float2 *src;
    float *dst;
    int32_t nd;
    int64_t total, total_k;
    int64_t ext[kExpandMaxD], stride[kExpandMaxD];
    float alpha_r, alpha_i;
    int32_t conj_x, conj_y;
};

__global__ void __launch_bounds__(256) complex_expand_kernel(const ComplexExpandParams p)
{
    const float s = p.conj_y ? -1.f : 1.f;
    for (int64_t e = int64_t(blockIdx.x) * blockDim.x + threadIdx.x; e < p.total; e += int64_t(gridDim.x) * blockDim.x) {
        int64_t lin = e, off = 0;
        for (int d = 0; d < p.nd; ++d) {
            const int64_t q = lin / p.ext[d];
            off += (lin - q * p.ext[d]) * p.stride[d];
            lin = q;
        }
        float2 x = p.src[off];
        if (p.conj_x) x.y = -x.y;
        const float xr = p.alpha_r * x.x - p.alpha_i * x.y, xi = p.alpha_r * x.y + p.alpha_i * x.x;
        const int64_t lin_k = e % p.total_k, lin_rest = e / p.total_k;
        float *o = p.dst + 2 * lin_k + 4 * p.total_k * lin_rest;
        *reinterpret_cast<float2 *>(o) = make_float2(xr, -s * xi);                     // v = 0: u = 0, 1
        *reinterpret_cast<float2 *>(o + 2 * p.total_k) = make_float2(xi, s * xr);      // v = 1
    }
}

}  // namespace btc

// Catch-all contraction kernel: correct for every legal input (any rank, signed or zero strides,
// repeated labels merged into summed strides, isolated labels of A or B summed as in Case 4).
// LANES threads cooperate on one element of D: they stride over the linearised summed index,
// reduce with warp shuffles, and lane 0 applies alpha/beta and stores through D's strides.
// Sums are kept in double (pairs for complex) for every element type.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"

namespace btc {

template <typename R> struct real_io;   // R = float or double; complex = 2 consecutive R
template <> struct real_io<float> { using type = float; };
template <> struct real_io<double> { using type = double; };

template <typename R, bool CPLX, int LANES>
__global__ void __launch_bounds__(256) generic_contract_kernel(const GenericParams p)
{
    constexpr int NC = CPLX ? 2 : 1;
    const R *A = static_cast<const R *>(p.A);
    const R *B = static_cast<const R *>(p.B);
    const R *C = static_cast<const R *>(p.C);
    R *D = static_cast<R *>(p.D);
    const int lane = (LANES == 1) ? 0 : int(threadIdx.x) % LANES;
    const int64_t group = (int64_t(blockIdx.x) * blockDim.x + threadIdx.x) / LANES;
    const int64_t ngroups = (int64_t(gridDim.x) * blockDim.x) / LANES;
    const double sa = p.conjA ? -1.0 : 1.0, sb = p.conjB ? -1.0 : 1.0, sc = p.conjC ? -1.0 : 1.0;

    for (int64_t e = group; e < p.total_d; e += ngroups) {
        int64_t offA = 0, offB = 0, offD = 0, lin = e;
        for (int d = 0; d < p.nd; ++d) {
            const int64_t i = lin % p.ext_d[d];
            lin /= p.ext_d[d];
            offA += i * p.sA_d[d];
            offB += i * p.sB_d[d];
            offD += i * p.sD_d[d];
        }
        double acc_r = 0.0, acc_i = 0.0;
        if (p.use_ab) {
            for (int64_t s = lane; s < p.total_k; s += LANES) {
                int64_t oa = offA, ob = offB, r = s;
                for (int d = 0; d < p.nk; ++d) {
                    const int64_t i = r % p.ext_k[d];
                    r /= p.ext_k[d];
                    oa += i * p.sA_k[d];
                    ob += i * p.sB_k[d];
                }
                if (!BTC_IN_SPAN(p.spans, 0, oa, 1) || !BTC_IN_SPAN(p.spans, 1, ob, 1)) continue;
                // a real operand among complex ones is read as (re, 0)
                const int na = p.cplxA ? 2 : 1, nb = p.cplxB ? 2 : 1;
                const double ar = double(A[na * oa]), br = double(B[nb * ob]);
                if (CPLX) {
                    const double ai = p.cplxA ? sa * double(A[na * oa + 1]) : 0.0;
                    const double bi = p.cplxB ? sb * double(B[nb * ob + 1]) : 0.0;
                    acc_r += ar * br - ai * bi;
                    acc_i += ar * bi + ai * br;
                } else {
                    acc_r += ar * br;
                }
            }
            if (LANES > 1) {
#pragma unroll
                for (int o = LANES / 2; o > 0; o >>= 1) {
                    acc_r += __shfl_xor_sync(0xffffffffu, acc_r, o);
                    if (CPLX) acc_i += __shfl_xor_sync(0xffffffffu, acc_i, o);
                }
            }
        }
        if (lane == 0 && BTC_IN_SPAN(p.spans, 2, offD, 1)) {
            double d_r = p.alpha[0] * acc_r - p.alpha[1] * acc_i;
            double d_i = p.alpha[0] * acc_i + p.alpha[1] * acc_r;
            if (p.use_c) {
                const int nc = p.cplxC ? 2 : 1;
                const double cr = double(C[nc * offD]);
                const double ci = p.cplxC ? sc * double(C[nc * offD + 1]) : 0.0;
                d_r += p.beta[0] * cr - p.beta[1] * ci;
                d_i += p.beta[0] * ci + p.beta[1] * cr;
            }
            D[NC * offD] = R(d_r);
            if (CPLX) D[NC * offD + (NC - 1)] = R(d_i);
        }
    }
}

}  // namespace btc

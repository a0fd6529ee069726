// Translation unit of the short-K streaming kernel for all element types (stream_kernel.cuh).
#include "stream_kernel.cuh"

#include "launchers.h"

namespace btc {

template <typename R, bool CPLX, int VFULL>
static cudaError_t launch_typed(const TiledParams &p, bool vec_d, bool vec_a, int sm_count, cudaStream_t st)
{
    const int64_t v = vec_d ? VFULL : 1;
    const int64_t total = ((p.M + v - 1) / v) * p.N * p.Bt;
    int64_t blocks = (total + kStreamThreads - 1) / kStreamThreads;
    const int64_t cap = int64_t(sm_count) * 32;            // grid-stride beyond 32 CTAs per SM
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    if (vec_d && VFULL > 1) {
        if (vec_a) stream_kernel<R, CPLX, VFULL, true><<<unsigned(blocks), kStreamThreads, 0, st>>>(p);
        else stream_kernel<R, CPLX, VFULL, false><<<unsigned(blocks), kStreamThreads, 0, st>>>(p);
    } else {
        stream_kernel<R, CPLX, 1, false><<<unsigned(blocks), kStreamThreads, 0, st>>>(p);
    }
    return cudaGetLastError();
}

cudaError_t launch_stream(const TiledParams &p, int dtype, bool vec_d, bool vec_a, int sm_count, cudaStream_t st)
{
    switch (dtype) {
    case 0: return launch_typed<float, false, 4>(p, vec_d, vec_a, sm_count, st);
    case 1: return launch_typed<double, false, 2>(p, vec_d, vec_a, sm_count, st);
    case 2: return launch_typed<float, true, 2>(p, vec_d, vec_a, sm_count, st);
    default: return launch_typed<double, true, 1>(p, vec_d, vec_a, sm_count, st);
    }
}

}  // namespace btc

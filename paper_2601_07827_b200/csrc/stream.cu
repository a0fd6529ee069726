// Translation unit of the short-K streaming kernel for all element types (stream_kernel.cuh).
#include "stream_kernel.cuh"

#include "launchers.h"

namespace btc {

template <typename R, bool CPLX, int VFULL>
static cudaError_t launch_typed(const TiledParams &p, bool vec_d, bool vec_a, cudaStream_t st)
{
    const int64_t v = vec_d ? VFULL : 1;
    const int64_t x_count = ((p.M + v - 1) / v) * p.Bt;
    int txv = 1;                                            // threads of a CTA along x: a power of two
    while (txv < kStreamThreads && txv < x_count) txv *= 2;
    const int64_t x_blocks = (x_count + txv - 1) / txv;
    const int64_t y_per_cta = int64_t(kStreamThreads / txv) * kStreamColumns;
    const int64_t blocks = x_blocks * ((p.N + y_per_cta - 1) / y_per_cta);
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (vec_d && VFULL > 1) {
        if (vec_a) stream_kernel<R, CPLX, VFULL, true><<<unsigned(blocks), kStreamThreads, 0, st>>>(p, txv, x_blocks);
        else stream_kernel<R, CPLX, VFULL, false><<<unsigned(blocks), kStreamThreads, 0, st>>>(p, txv, x_blocks);
    } else {
        stream_kernel<R, CPLX, 1, false><<<unsigned(blocks), kStreamThreads, 0, st>>>(p, txv, x_blocks);
    }
    return cudaGetLastError();
}

cudaError_t launch_stream(const TiledParams &p, int dtype, bool vec_d, bool vec_a, int /*sm_count*/, cudaStream_t st)
{
    switch (dtype) {
    case 0: return launch_typed<float, false, 4>(p, vec_d, vec_a, st);
    case 1: return launch_typed<double, false, 2>(p, vec_d, vec_a, st);
    case 2: return launch_typed<float, true, 2>(p, vec_d, vec_a, st);
    default: return launch_typed<double, true, 1>(p, vec_d, vec_a, st);
    }
}

}  // namespace btc

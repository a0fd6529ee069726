// Transpose-free tiled contraction kernel for fp32 on the FP32 FMA pipe (sm_100a).
//
// Same structure as the fp64 kernel: a producer warpgroup gathers strided BM x BK / BK x BN
// tiles of A and B with cp.async into whichever shared-memory orientation matches the operand's
// contiguous direction, consumer warps do the arithmetic, mbarriers hand stages over.  The
// consumers keep a TM x TN register tile per thread.  An operand stored with the free index
// contiguous is read one k at a time as 16-byte vectors over 4 consecutive rows; an operand
// stored with k contiguous is read 4 k at a time, one 16-byte vector per row, with the rows of a
// thread interleaved (row = lane row + 8 i) so that the vector loads of a quarter warp fall into
// distinct banks.  Both orientations therefore cost the same number of shared-memory loads per
// FMA, and neither needs a transposed copy of the operand.
#pragma once

#include <cuda_runtime.h>

#include "epilogue_common.cuh"
#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

template <int BM_, int BN_, int BK_, int WARPS_M_, int WARPS_N_, int STAGES_, int MIN_CTAS_, bool PREFETCH_>
struct F32Tile {
    static constexpr int BM = BM_, BN = BN_, BK = BK_;
    static constexpr bool PREFETCH = PREFETCH_;
    static constexpr int WARPS_M = WARPS_M_, WARPS_N = WARPS_N_;
    static constexpr int CONSUMER_WARPS = WARPS_M_ * WARPS_N_;
    static constexpr int CONSUMER_THREADS = 32 * CONSUMER_WARPS;
    static constexpr int PRODUCER_THREADS = 32 * kProducerWarps;
    static constexpr int THREADS = CONSUMER_THREADS + PRODUCER_THREADS;
    static constexpr int MIN_CTAS = MIN_CTAS_;
    static constexpr bool REBALANCE_REGS = (THREADS == 384 && MIN_CTAS_ == 1);
    static constexpr int STAGES = STAGES_;
    static constexpr int WM = BM / WARPS_M, WN = BN / WARPS_N;
    static constexpr int TM = WM / 8, TN = WN / 4;    // a warp is 8 (rows) x 4 (columns) threads
    static constexpr int ACC = TM * TN;
    static_assert(TM % 4 == 0 && TN % 4 == 0, "register tile must be made of 4-vectors");
    // pitches in floats: multiples of 4 (16-byte vectors); the k-contiguous pitch 20 puts the
    // 8 (or 4) rows a quarter warp reads into distinct banks
    static constexpr int PITCH_FREE_A = BM + 4, PITCH_FREE_B = BN + 4, PITCH_K = BK + 4;
    static constexpr int A_ELEMS = (BK * PITCH_FREE_A > BM * PITCH_K) ? BK * PITCH_FREE_A : BM * PITCH_K;
    static constexpr int B_ELEMS = (BK * PITCH_FREE_B > BN * PITCH_K) ? BK * PITCH_FREE_B : BN * PITCH_K;
    static constexpr int STAGE_FLOATS = A_ELEMS + B_ELEMS;
    static constexpr size_t IMAGE_BYTES = size_t(BN) * (BM + 4) * 4;        // epilogue image of the tile
    static constexpr size_t STAGES_BYTES = size_t(STAGES) * STAGE_FLOATS * 4;
    static constexpr size_t SMEM_BYTES =
        (STAGES_BYTES > IMAGE_BYTES ? STAGES_BYTES : IMAGE_BYTES) + size_t(2 * BM + 2 * BN + 2 * kKoffCap) * 8 + size_t(2 * STAGES) * 8 + 16;
};

// tile-local row of register-tile entry i (and column of entry j) for the two orientations
template <bool KMAJ> __device__ __forceinline__ int f32_row_of(int ty, int i)
{
    return KMAJ ? ty + 8 * i : (i >> 2) * 32 + ty * 4 + (i & 3);
}
template <bool KMAJ> __device__ __forceinline__ int f32_col_of(int tx, int j)
{
    return KMAJ ? tx + 4 * j : (j >> 2) * 16 + tx * 4 + (j & 3);
}

template <typename T, bool A_KMAJ, bool B_KMAJ>
__global__ void __launch_bounds__(T::THREADS, T::MIN_CTAS) tiled_f32_kernel(const TiledParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *stage_base = reinterpret_cast<float *>(smem_raw);
    int64_t *rowA = reinterpret_cast<int64_t *>(smem_raw + (T::STAGES_BYTES > T::IMAGE_BYTES ? T::STAGES_BYTES : T::IMAGE_BYTES));
    int64_t *rowD = rowA + T::BM;
    int64_t *colB = rowD + T::BM;
    int64_t *colD = colB + T::BN;
    int64_t *koffA = colD + T::BN;
    int64_t *koffB = koffA + kKoffCap;
    uint64_t *bars = reinterpret_cast<uint64_t *>(koffB + kKoffCap);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * T::STAGES);
    const unsigned full0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned empty0 = full0 + 8u * T::STAGES;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileCoords tc = tile_coords<T::BM, T::BN, T::BK>(p);
    tile_setup<T::BM, T::BN, T::STAGES, T::THREADS, T::PRODUCER_THREADS, T::CONSUMER_WARPS>(
        p, tc, rowA, rowD, colB, colD, koffA, koffB, full0, empty0, abort_flag, tid);

    constexpr int a_srow = A_KMAJ ? T::PITCH_K : 1, a_sk = A_KMAJ ? 1 : T::PITCH_FREE_A;
    constexpr int b_srow = B_KMAJ ? T::PITCH_K : 1, b_sk = B_KMAJ ? 1 : T::PITCH_FREE_B;

    if (warp < kProducerWarps) {
        if (T::REBALANCE_REGS) reg_dec<40>();
        const unsigned stage0 = static_cast<unsigned>(__cvta_generic_to_shared(stage_base));
        producer_loop<T::BM, T::BN, T::BK, 4, T::STAGES, T::STAGE_FLOATS * 4, T::A_ELEMS * 4, T::PRODUCER_THREADS>(
            p, tc, stage0, rowA, colB, koffA, koffB, full0, empty0, abort_flag, a_srow, a_sk, b_srow, b_sk, tid);
        return;
    }

    if (T::REBALANCE_REGS) reg_inc<232>();
    const int cw = warp - kProducerWarps;
    const int ctid = tid - T::PRODUCER_THREADS;
    const int wm0 = (cw % T::WARPS_M) * T::WM, wn0 = (cw / T::WARPS_M) * T::WN;
    const int ty = lane >> 2, tx = lane & 3;

    float acc[T::TM][T::TN];
#pragma unroll
    for (int i = 0; i < T::TM; ++i)
#pragma unroll
        for (int j = 0; j < T::TN; ++j) acc[i][j] = 0.f;

    bool ok = true;
    for (int kt = 0; kt < tc.num_kt; ++kt) {
        const int s = kt % T::STAGES, round = kt / T::STAGES;
        if (!mbar_wait_bounded(full0 + 8u * s, unsigned(round) & 1u, abort_flag, p.error_word, kErrFullWait, p.poll_limit)) {
            ok = false;
            break;
        }
        const float *sa = stage_base + size_t(s) * T::STAGE_FLOATS;
        const float *sb = sa + T::A_ELEMS;
        // fragments of 4 consecutive k live in registers; with PREFETCH the next group's loads
        // are issued before the current group's FMAs
        float fa[T::PREFETCH ? 2 : 1][T::TM][4], fb[T::PREFETCH ? 2 : 1][T::TN][4];
        auto load_group = [&](int buf, int k4) {
            if (A_KMAJ) {
#pragma unroll
                for (int i = 0; i < T::TM; ++i) {
                    const float4 v = *reinterpret_cast<const float4 *>(sa + (wm0 + ty + 8 * i) * T::PITCH_K + k4);
                    fa[buf][i][0] = v.x; fa[buf][i][1] = v.y; fa[buf][i][2] = v.z; fa[buf][i][3] = v.w;
                }
            } else {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                    for (int i4 = 0; i4 < T::TM / 4; ++i4) {
                        const float4 v = *reinterpret_cast<const float4 *>(
                            sa + (k4 + kk) * T::PITCH_FREE_A + wm0 + i4 * 32 + ty * 4);
                        fa[buf][i4 * 4][kk] = v.x; fa[buf][i4 * 4 + 1][kk] = v.y;
                        fa[buf][i4 * 4 + 2][kk] = v.z; fa[buf][i4 * 4 + 3][kk] = v.w;
                    }
            }
            if (B_KMAJ) {
#pragma unroll
                for (int j = 0; j < T::TN; ++j) {
                    const float4 v = *reinterpret_cast<const float4 *>(sb + (wn0 + tx + 4 * j) * T::PITCH_K + k4);
                    fb[buf][j][0] = v.x; fb[buf][j][1] = v.y; fb[buf][j][2] = v.z; fb[buf][j][3] = v.w;
                }
            } else {
#pragma unroll
                for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                    for (int j4 = 0; j4 < T::TN / 4; ++j4) {
                        const float4 v = *reinterpret_cast<const float4 *>(
                            sb + (k4 + kk) * T::PITCH_FREE_B + wn0 + j4 * 16 + tx * 4);
                        fb[buf][j4 * 4][kk] = v.x; fb[buf][j4 * 4 + 1][kk] = v.y;
                        fb[buf][j4 * 4 + 2][kk] = v.z; fb[buf][j4 * 4 + 3][kk] = v.w;
                    }
            }
        };
        if (T::PREFETCH) load_group(0, 0);
#pragma unroll
        for (int g = 0; g < T::BK / 4; ++g) {
            const int cur = T::PREFETCH ? (g & 1) : 0;
            if (!T::PREFETCH) load_group(0, g * 4);
            else if (g + 1 < T::BK / 4) load_group(cur ^ 1, (g + 1) * 4);
#pragma unroll
            for (int kk = 0; kk < 4; ++kk)
#pragma unroll
                for (int i = 0; i < T::TM; ++i)
#pragma unroll
                    for (int j = 0; j < T::TN; ++j) acc[i][j] = fmaf(fa[cur][i][kk], fb[cur][j][kk], acc[i][j]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * s);
    }
    (void)ok;   // a wait that gave up has raised the CTA's abort flag

    // Epilogue: register tile -> image of the CTA tile in the idle stage buffers -> rolled walk.
    consumer_barrier<T::CONSUMER_THREADS>();
    if (*abort_flag) return;
    float *image = stage_base;
    constexpr int P = ImagePitch<T::BM>::value;
#pragma unroll
    for (int j = 0; j < T::TN; ++j) {
        const int c = wn0 + f32_col_of<B_KMAJ>(tx, j);
#pragma unroll
        for (int i = 0; i < T::TM; ++i) image[c * P + wm0 + f32_row_of<A_KMAJ>(ty, i)] = acc[i][j];
    }
    consumer_barrier<T::CONSUMER_THREADS>();
    store_tile_image<float, 1, T::BM, T::BN, T::CONSUMER_THREADS>(p, tc, image, rowD, colD, ctid);
}

}  // namespace btc

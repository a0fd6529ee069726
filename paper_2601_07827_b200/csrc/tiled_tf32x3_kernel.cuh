// Tensor-core tiled contraction kernel for fp32 and complex64 on sm_100a: 3xTF32.
//
// Every fp32 operand is split in registers into a TF32 head and a TF32 tail (x = hi + lo with
// hi = x cut to TF32, lo = x - hi, exact in fp32), and each product runs as three tensor-core
// MMAs, lo*hi + hi*lo + hi*hi, accumulated in fp32.  The dropped lo*lo term and the cut of lo are
// each about 2^-20 relative to |a||b|, far inside the 1e-5 tolerance of the fp32 types;
// inputs that are exactly representable in TF32 (small integers) give exact products.
//
// Structure as in the fp64 kernel: a producer warpgroup gathers strided tiles with cp.async in
// whichever orientation matches each operand, consumer warps read m16n8k8 fragments word by word
// (so either orientation works, with pitches chosen conflict-free), mbarriers hand stages over.
// Complex64 uses the real expansion [[br, sb*bi], [-sa*sb*bi, sa*br]] at fragment load, so one
// accumulator fragment holds 4 complex columns with (re, im) adjacent.
#pragma once

#include <cuda_runtime.h>

#include "epilogue_common.cuh"
#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

template <bool CPLX_, int BM_, int BN_, int WARPS_M_, int WARPS_N_, int STAGES_, int MIN_CTAS_>
struct TF32Tile {
    static constexpr bool CPLX = CPLX_;
    static constexpr int BM = BM_, BN = BN_;          // elements
    static constexpr int BK = CPLX_ ? 16 : 32;        // elements per stage (32 real k either way)
    static constexpr int W = CPLX_ ? 2 : 1;           // 4-byte words per element
    static constexpr int WARPS_M = WARPS_M_, WARPS_N = WARPS_N_;
    static constexpr int CONSUMER_WARPS = WARPS_M_ * WARPS_N_;
    static constexpr int CONSUMER_THREADS = 32 * CONSUMER_WARPS;
    static constexpr int PRODUCER_THREADS = 32 * kProducerWarps;
    static constexpr int THREADS = CONSUMER_THREADS + PRODUCER_THREADS;
    static constexpr int MIN_CTAS = MIN_CTAS_;
    static constexpr bool REBALANCE_REGS = (THREADS == 384 && MIN_CTAS_ == 1);
    static constexpr int STAGES = STAGES_;
    static constexpr int WM = BM / WARPS_M;           // warp tile rows
    static constexpr int WNR = BN * W / WARPS_N;      // warp tile columns in real words
    static constexpr int FM = WM / 16, FN = WNR / 8;  // m16n8 fragments per warp
    static constexpr int ACC = FM * FN * 4;           // floats per consumer thread
    // pitches in elements, conflict-free for word-wise fragment reads:
    //   real: free-index pitch = 8 (mod 32), k pitch = 4 (mod 32) or 20
    //   complex: free-index pitch = 8 (mod 16), k pitch = 2 (mod 16)
    static constexpr int PITCH_FREE_A = BM + 8, PITCH_FREE_B = BN + 8;
    static constexpr int PITCH_K = CPLX_ ? BK + 2 : BK + 4;
    static constexpr int A_ELEMS = (BK * PITCH_FREE_A > BM * PITCH_K) ? BK * PITCH_FREE_A : BM * PITCH_K;
    static constexpr int B_ELEMS = (BK * PITCH_FREE_B > BN * PITCH_K) ? BK * PITCH_FREE_B : BN * PITCH_K;
    static constexpr int STAGE_WORDS = (A_ELEMS + B_ELEMS) * W;
    static constexpr size_t IMAGE_BYTES = size_t(BN) * (BM + 4) * W * 4;    // epilogue image of the tile
    static constexpr size_t STAGES_BYTES = size_t(STAGES) * STAGE_WORDS * 4;
    static constexpr size_t SMEM_BYTES =
        (STAGES_BYTES > IMAGE_BYTES ? STAGES_BYTES : IMAGE_BYTES) + size_t(2 * BM + 2 * BN + 2 * kKoffCap) * 8 + size_t(2 * STAGES) * 8 + 16;
};

__device__ __forceinline__ void mma_tf32_m16n8k8(float (&c)[4], const unsigned (&a)[4], const unsigned (&b)[2])
{
    asm volatile("mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
}

// x = hi + lo with hi = x cut to TF32 (the top 10 mantissa bits) and lo = x - hi, which is exact
// in fp32 and holds the remaining 13 bits; cutting lo to TF32 as well drops at most 2^-21 |x|.
__device__ __forceinline__ void split_tf32(float x, unsigned &hi, unsigned &lo)
{
    hi = __float_as_uint(x) & 0xffffe000u;
    lo = __float_as_uint(x - __uint_as_float(hi)) & 0xffffe000u;
}

template <typename T>
__global__ void __launch_bounds__(T::THREADS, T::MIN_CTAS) tiled_tf32x3_kernel(const TiledParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int W = T::W;
    constexpr int EB = 4 * W;
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

    const int a_srow = p.dirA == 0 ? 1 : T::PITCH_K, a_sk = p.dirA == 0 ? T::PITCH_FREE_A : 1;
    const int b_srow = p.dirB == 0 ? 1 : T::PITCH_K, b_sk = p.dirB == 0 ? T::PITCH_FREE_B : 1;

    if (warp < kProducerWarps) {
        if (T::REBALANCE_REGS) reg_dec<40>();
        const unsigned stage0 = static_cast<unsigned>(__cvta_generic_to_shared(stage_base));
        producer_loop<T::BM, T::BN, T::BK, EB, T::STAGES, T::STAGE_WORDS * 4, T::A_ELEMS * EB, T::PRODUCER_THREADS>(
            p, tc, stage0, rowA, colB, koffA, koffB, full0, empty0, abort_flag, a_srow, a_sk, b_srow, b_sk, tid);
        return;
    }

    if (T::REBALANCE_REGS) reg_inc<232>();
    const int cw = warp - kProducerWarps;
    const int ctid = tid - T::PRODUCER_THREADS;
    const int wm0 = (cw % T::WARPS_M) * T::WM;
    const int wn0w = (cw / T::WARPS_M) * T::WNR;
    const int g = lane >> 2, t = lane & 3;

    // word offsets inside a stage of this lane's fragment entries:
    //   A: a0 (row g, k t), a1 (row g+8, k t), a2 (row g, k t+4), a3 (row g+8, k t+4)
    //   B: b0 (k t, col g), b1 (k t+4, col g)
    int a_thr, a_row8, a_k4, a_istep, a_kstep, b_thr, b_k4, b_jstep, b_kstep;
    unsigned b_sign = 0;
    if (!T::CPLX) {
        a_thr = (wm0 + g) * a_srow + t * a_sk;
        a_row8 = 8 * a_srow;  a_k4 = 4 * a_sk;  a_istep = 16 * a_srow;  a_kstep = 8 * a_sk;
        b_thr = (wn0w + g) * b_srow + t * b_sk;
        b_k4 = 4 * b_sk;  b_jstep = 8 * b_srow;  b_kstep = 8 * b_sk;
    } else {
        const int pbit = t & 1, qbit = g & 1;
        a_thr = ((wm0 + g) * a_srow + (t >> 1) * a_sk) * 2 + pbit;
        a_row8 = 16 * a_srow;  a_k4 = 4 * a_sk;  a_istep = 32 * a_srow;  a_kstep = 8 * a_sk;
        b_thr = ((wn0w / 2 + (g >> 1)) * b_srow + (t >> 1) * b_sk) * 2 + (pbit ^ qbit);
        b_k4 = 4 * b_sk;  b_jstep = 8 * b_srow;  b_kstep = 8 * b_sk;
        // block [[br, sb*bi], [-sa*sb*bi, sa*br]]: entry (p, q) is negative when
        //   (0,1): sb < 0;  (1,0): sa*sb > 0;  (1,1): sa < 0
        const bool na = p.conjA != 0, nb = p.conjB != 0;
        bool neg = false;
        if (pbit == 0 && qbit == 1) neg = nb;
        if (pbit == 1 && qbit == 0) neg = (na == nb);
        if (pbit == 1 && qbit == 1) neg = na;
        b_sign = neg ? 0x80000000u : 0u;
    }

    float acc[T::FM][T::FN][4];
#pragma unroll
    for (int i = 0; i < T::FM; ++i)
#pragma unroll
        for (int j = 0; j < T::FN; ++j)
#pragma unroll
            for (int c = 0; c < 4; ++c) acc[i][j][c] = 0.f;

    bool ok = true;
    for (int kt = 0; kt < tc.num_kt; ++kt) {
        const int s = kt % T::STAGES, round = kt / T::STAGES;
        if (!mbar_wait_bounded(full0 + 8u * s, unsigned(round) & 1u, abort_flag, p.error_word, kErrFullWait, p.poll_limit)) {
            ok = false;
            break;
        }
        const float *sa = stage_base + size_t(s) * T::STAGE_WORDS;
        const float *sb = sa + T::A_ELEMS * W;
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {          // 32 real k per stage, 8 per MMA
            unsigned a_hi[T::FM][4], a_lo[T::FM][4], b_hi[T::FN][2], b_lo[T::FN][2];
#pragma unroll
            for (int i = 0; i < T::FM; ++i) {
                const float *pa = sa + a_thr + i * a_istep + kk * a_kstep;
                split_tf32(pa[0], a_hi[i][0], a_lo[i][0]);
                split_tf32(pa[a_row8], a_hi[i][1], a_lo[i][1]);
                split_tf32(pa[a_k4], a_hi[i][2], a_lo[i][2]);
                split_tf32(pa[a_row8 + a_k4], a_hi[i][3], a_lo[i][3]);
            }
#pragma unroll
            for (int j = 0; j < T::FN; ++j) {
                const float *pb = sb + b_thr + j * b_jstep + kk * b_kstep;
                float v0 = pb[0], v1 = pb[b_k4];
                if (T::CPLX) {
                    v0 = __uint_as_float(__float_as_uint(v0) ^ b_sign);
                    v1 = __uint_as_float(__float_as_uint(v1) ^ b_sign);
                }
                split_tf32(v0, b_hi[j][0], b_lo[j][0]);
                split_tf32(v1, b_hi[j][1], b_lo[j][1]);
            }
#pragma unroll
            for (int i = 0; i < T::FM; ++i)
#pragma unroll
                for (int j = 0; j < T::FN; ++j) {
                    mma_tf32_m16n8k8(acc[i][j], a_lo[i], b_hi[j]);
                    mma_tf32_m16n8k8(acc[i][j], a_hi[i], b_lo[j]);
                    mma_tf32_m16n8k8(acc[i][j], a_hi[i], b_hi[j]);
                }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * s);
    }
    (void)ok;   // a wait that gave up has raised the CTA's abort flag

    // Epilogue: fragments -> image of the tile in the idle stage buffers -> rolled walk.
    // Fragment (fi, fj): c0, c1 -> row g, columns 2t, 2t+1; c2, c3 -> row g+8, same columns.
    consumer_barrier<T::CONSUMER_THREADS>();
    if (*abort_flag) return;
    float *image = stage_base;
    constexpr int P = ImagePitch<T::BM>::value;
#pragma unroll
    for (int fi = 0; fi < T::FM; ++fi)
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            const int r = wm0 + fi * 16 + half * 8 + g;
#pragma unroll
            for (int fj = 0; fj < T::FN; ++fj) {
                const float v0 = acc[fi][fj][half * 2], v1 = acc[fi][fj][half * 2 + 1];
                if (T::CPLX) {
                    const int c = (wn0w + fj * 8) / 2 + t;
                    *reinterpret_cast<float2 *>(image + size_t(c * P + r) * 2) = make_float2(v0, v1);
                } else {
                    const int c = wn0w + fj * 8 + 2 * t;
                    image[c * P + r] = v0;
                    image[(c + 1) * P + r] = v1;
                }
            }
        }
    consumer_barrier<T::CONSUMER_THREADS>();
    store_tile_image<float, W, T::BM, T::BN, T::CONSUMER_THREADS>(p, tc, image, rowD, colD, ctid);
}

}  // namespace btc

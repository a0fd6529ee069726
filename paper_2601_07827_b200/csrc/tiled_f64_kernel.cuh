// Transpose-free tiled contraction kernel for fp64 and complex128 on sm_100a.
//
// The three linearised indices m (free labels of A), n (free labels of B) and k (contracted
// labels) address memory through per-index offset tables, so a CTA gathers a BM x BK tile of
// op(A) and a BK x BN tile of op(B) straight from the strided tensors into shared memory with
// cp.async (16-byte copies where the strides allow, element copies otherwise), in whichever
// direction is closest to contiguous for that operand, and keeps that orientation in shared
// memory: the FP64 tensor-core fragments (mma.sync m8n8k4, one 8-byte word per lane) can be read
// from either orientation without bank conflicts, so no transpose is ever materialised.
//
// The CTA is warp-specialised: one warpgroup of producer warps does all address arithmetic and
// issues the cp.async gathers; the consumer warps only read fragments and issue MMAs.  The two
// sides hand shared-memory stages to each other through mbarriers ("full": armed by the
// completion of the producers' copies; "empty": one arrival per consumer warp).  Every wait is
// bounded: when a wait runs out the kernel records an error word, raises a CTA-wide abort flag
// so the other waits end too, drains its copies and returns.
//
// Complex128 runs on the same real MMAs: an interleaved (re, im) row of A is a real row of
// twice the length, and each complex b expands at fragment-load time into the 2x2 real block
// [[br, sb*bi], [-sa*sb*bi, sa*br]] (sa, sb = -1 when that operand is conjugated), which gives
// exactly 8 real flops per complex multiply-add.  An 8x8 accumulator fragment then holds
// 8 rows x 4 complex columns with (re, im) adjacent in one lane.
//
// With split-K each CTA handles one slice of k and stores raw accumulators to scratch; a second
// kernel adds the slices in a fixed order and applies alpha/beta, so results do not depend on
// scheduling.
#pragma once

#include <cuda_runtime.h>

#include "epilogue_common.cuh"
#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

template <bool CPLX_, int BM_, int BN_, int WARPS_M_, int WARPS_N_, int STAGES_, int MIN_CTAS_, bool MMA16_ = false>
struct F64Tile {
    static constexpr bool CPLX = CPLX_;
    static constexpr bool MMA16 = MMA16_;             // one m16n8k16 MMA per stage instead of m8n8k4 steps
    static constexpr int BM = BM_;                    // rows of the CTA tile (elements)
    static constexpr int BN = BN_;                    // columns of the CTA tile (elements)
    static constexpr int BK = CPLX_ ? 8 : 16;         // k extent of one stage (elements)
    static constexpr int W = CPLX_ ? 2 : 1;           // 8-byte words per element
    static constexpr int WARPS_M = WARPS_M_, WARPS_N = WARPS_N_;
    static constexpr int CONSUMER_WARPS = WARPS_M_ * WARPS_N_;
    static constexpr int CONSUMER_THREADS = 32 * CONSUMER_WARPS;
    static constexpr int PRODUCER_THREADS = 32 * kProducerWarps;
    static constexpr int THREADS = CONSUMER_THREADS + PRODUCER_THREADS;
    static constexpr int MIN_CTAS = MIN_CTAS_;
    // with 12 warps the register file gives 168 registers per thread; the consumers need more,
    // the producers far fewer, so the warpgroups re-split the file (setmaxnreg)
    static constexpr bool REBALANCE_REGS = (THREADS == 384 && MIN_CTAS_ == 1);
    static constexpr int STAGES = STAGES_;
    static constexpr int WM = BM / WARPS_M;           // warp tile rows
    static constexpr int WNR = BN * W / WARPS_N;      // warp tile columns in real words
    static constexpr int FM = WM / 8, FN = WNR / 8;   // 8x8 fragments per warp
    static constexpr int ACC = FM * FN * 2;           // doubles per consumer thread
    // shared-memory pitches (elements): conflict-free fragment reads need
    //   real:    pitch = 4 (mod 16);   complex: pitch = 4 (mod 8) along the free index,
    //                                           pitch = 2 (mod 8) along k
    static constexpr int PITCH_FREE_A = BM + 4, PITCH_FREE_B = BN + 4;
    static constexpr int PITCH_K = CPLX_ ? BK + 2 : BK + 4;
    static constexpr int A_ELEMS = (BK * PITCH_FREE_A > BM * PITCH_K) ? BK * PITCH_FREE_A : BM * PITCH_K;
    static constexpr int B_ELEMS = (BK * PITCH_FREE_B > BN * PITCH_K) ? BK * PITCH_FREE_B : BN * PITCH_K;
    static constexpr int STAGE_WORDS = (A_ELEMS + B_ELEMS) * W;
    // stages | row/column offset arrays | full[STAGES], empty[STAGES] mbarriers | abort flag
    static constexpr size_t IMAGE_BYTES = size_t(BN) * (BM + 4) * W * 8;    // epilogue image of the tile
    static constexpr size_t STAGES_BYTES = size_t(STAGES) * STAGE_WORDS * 8;
    static constexpr size_t SMEM_BYTES =
        (STAGES_BYTES > IMAGE_BYTES ? STAGES_BYTES : IMAGE_BYTES) + size_t(2 * BM + 2 * BN + 2 * kKoffCap) * 8 + size_t(2 * STAGES) * 8 + 16;
};

// m16n8k16: A rows g / g+8 (even / odd register), k = t + 4 (i / 2); B k = t + 4 j, column g;
// C rows g (c0, c1) and g + 8 (c2, c3), columns 2t, 2t + 1
__device__ __forceinline__ void dmma_m16n8k16(double (&c)[4], const double (&a)[8], const double (&b)[4])
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f64.f64.f64.f64 {%0,%1,%2,%3}, {%4,%5,%6,%7,%8,%9,%10,%11}, "
                 "{%12,%13,%14,%15}, {%0,%1,%2,%3};"
                 : "+d"(c[0]), "+d"(c[1]), "+d"(c[2]), "+d"(c[3])
                 : "d"(a[0]), "d"(a[1]), "d"(a[2]), "d"(a[3]), "d"(a[4]), "d"(a[5]), "d"(a[6]), "d"(a[7]),
                   "d"(b[0]), "d"(b[1]), "d"(b[2]), "d"(b[3]));
}

__device__ __forceinline__ void dmma_m8n8k4(double &c0, double &c1, double a, double b)
{
    asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
                 : "+d"(c0), "+d"(c1) : "d"(a), "d"(b));
}

template <typename T>
__global__ void __launch_bounds__(T::THREADS, T::MIN_CTAS) tiled_f64_kernel(const TiledParams p)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    constexpr int W = T::W;
    constexpr int EB = 8 * W;
    double *stage_base = reinterpret_cast<double *>(smem_raw);
    int64_t *rowA = reinterpret_cast<int64_t *>(smem_raw + (T::STAGES_BYTES > T::IMAGE_BYTES ? T::STAGES_BYTES : T::IMAGE_BYTES));
    int64_t *rowD = rowA + T::BM;
    int64_t *colB = rowD + T::BM;
    int64_t *colD = colB + T::BN;
    int64_t *koffA = colD + T::BN;
    int64_t *koffB = koffA + kKoffCap;
    uint64_t *bars = reinterpret_cast<uint64_t *>(koffB + kKoffCap);      // full[STAGES], empty[STAGES]
    volatile int *abort_flag = reinterpret_cast<volatile int *>(bars + 2 * T::STAGES);
    const unsigned full0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned empty0 = full0 + 8u * T::STAGES;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileCoords tc = tile_coords<T::BM, T::BN, T::BK>(p);
    const int rows_valid = tc.rows_valid, cols_valid = tc.cols_valid, num_kt = tc.num_kt;
    (void)rows_valid; (void)cols_valid;
    tile_setup<T::BM, T::BN, T::STAGES, T::THREADS, T::PRODUCER_THREADS, T::CONSUMER_WARPS>(
        p, tc, rowA, rowD, colB, colD, koffA, koffB, full0, empty0, abort_flag, tid);

    // shared-memory orientation follows the load direction of each operand
    const int a_srow = p.dirA == 0 ? 1 : T::PITCH_K, a_sk = p.dirA == 0 ? T::PITCH_FREE_A : 1;
    const int b_srow = p.dirB == 0 ? 1 : T::PITCH_K, b_sk = p.dirB == 0 ? T::PITCH_FREE_B : 1;

    if (warp < kProducerWarps) {
        // ------------------------------------------------------------------ producers
        if (T::REBALANCE_REGS) reg_dec<40>();
        const unsigned stage0 = static_cast<unsigned>(__cvta_generic_to_shared(stage_base));
        producer_loop<T::BM, T::BN, T::BK, EB, T::STAGES, T::STAGE_WORDS * 8, T::A_ELEMS * EB, T::PRODUCER_THREADS>(
            p, tc, stage0, rowA, colB, koffA, koffB, full0, empty0, abort_flag, a_srow, a_sk, b_srow, b_sk, tid);
        return;
    }

    // ---------------------------------------------------------------------- consumers
    if (T::REBALANCE_REGS) reg_inc<232>();
    const int cw = warp - kProducerWarps;
    const int ctid = tid - T::PRODUCER_THREADS;
    const int warp_m = cw % T::WARPS_M, warp_n = cw / T::WARPS_M;
    const int wm0 = warp_m * T::WM;
    const int wn0w = warp_n * T::WNR;            // first real-word column of the warp tile
    const int g = lane >> 2, t = lane & 3;

    // word offsets of this lane's fragment entries inside a stage
    int a_thr, a_istep, a_kstep, b_thr, b_jstep, b_kstep;
    unsigned b_sign = 0;                         // xor mask for the high word of b
    if (!T::CPLX) {
        a_thr = (wm0 + g) * a_srow + t * a_sk;
        a_istep = 8 * a_srow;
        a_kstep = 4 * a_sk;
        b_thr = (wn0w + g) * b_srow + t * b_sk;
        b_jstep = 8 * b_srow;
        b_kstep = 4 * b_sk;
    } else {
        const int pbit = t & 1, qbit = g & 1;
        a_thr = ((wm0 + g) * a_srow + (t >> 1) * a_sk) * 2 + pbit;
        a_istep = 16 * a_srow;
        a_kstep = 4 * a_sk;
        b_thr = ((wn0w / 2 + (g >> 1)) * b_srow + (t >> 1) * b_sk) * 2 + (pbit ^ qbit);
        b_jstep = 8 * b_srow;
        b_kstep = 4 * b_sk;
        // block [[br, sb*bi], [-sa*sb*bi, sa*br]]: entry (p, q) is negative when
        //   (0,1): sb < 0;  (1,0): sa*sb > 0;  (1,1): sa < 0
        const bool na = p.conjA != 0, nb = p.conjB != 0;
        bool neg = false;
        if (pbit == 0 && qbit == 1) neg = nb;
        if (pbit == 1 && qbit == 0) neg = (na == nb);
        if (pbit == 1 && qbit == 1) neg = na;
        b_sign = neg ? 0x80000000u : 0u;
    }

    double acc[T::FM][T::FN][2];
#pragma unroll
    for (int i = 0; i < T::FM; ++i)
#pragma unroll
        for (int j = 0; j < T::FN; ++j) acc[i][j][0] = acc[i][j][1] = 0.0;

    bool ok = true;
    for (int kt = 0; kt < num_kt; ++kt) {
        const int s = kt % T::STAGES, round = kt / T::STAGES;
        if (!mbar_wait_bounded(full0 + 8u * s, unsigned(round) & 1u, abort_flag, p.error_word, kErrFullWait, p.poll_limit)) {
            ok = false;
            break;
        }
        const double *sa = stage_base + size_t(s) * T::STAGE_WORDS;
        const double *sb = sa + T::A_ELEMS * W;
        if (T::MMA16) {
            // acc[2 i2][j] / acc[2 i2 + 1][j] are the row halves g / g + 8 of a 16-row fragment
#pragma unroll
            for (int half = 0; half < 2; ++half) {       // limits live fragment registers
                double a16[T::FM / 4][8], b16[T::FN][4];
#pragma unroll
                for (int j = 0; j < T::FN; ++j)
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        double b = sb[b_thr + j * b_jstep + q * b_kstep];
                        if (T::CPLX) {
                            int hi = __double2hiint(b) ^ int(b_sign);
                            b = __hiloint2double(hi, __double2loint(b));
                        }
                        b16[j][q] = b;
                    }
#pragma unroll
                for (int i2 = 0; i2 < T::FM / 4; ++i2)
#pragma unroll
                    for (int r = 0; r < 8; ++r)
                        a16[i2][r] = sa[a_thr + ((half * (T::FM / 4) + i2) * 2 + (r & 1)) * a_istep + (r >> 1) * a_kstep];
#pragma unroll
                for (int i2 = 0; i2 < T::FM / 4; ++i2)
#pragma unroll
                    for (int j = 0; j < T::FN; ++j) {
                        const int i = (half * (T::FM / 4) + i2) * 2;
                        double c[4] = {acc[i][j][0], acc[i][j][1], acc[i + 1][j][0], acc[i + 1][j][1]};
                        dmma_m16n8k16(c, a16[i2], b16[j]);
                        acc[i][j][0] = c[0]; acc[i][j][1] = c[1]; acc[i + 1][j][0] = c[2]; acc[i + 1][j][1] = c[3];
                    }
            }
        } else
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {         // 16 real k per stage, 4 per MMA
            double af[T::FM], bf[T::FN];
#pragma unroll
            for (int i = 0; i < T::FM; ++i) af[i] = sa[a_thr + i * a_istep + kk * a_kstep];
#pragma unroll
            for (int j = 0; j < T::FN; ++j) {
                double b = sb[b_thr + j * b_jstep + kk * b_kstep];
                if (T::CPLX) {
                    int hi = __double2hiint(b) ^ int(b_sign);
                    b = __hiloint2double(hi, __double2loint(b));
                }
                bf[j] = b;
            }
#pragma unroll
            for (int i = 0; i < T::FM; ++i)
#pragma unroll
                for (int j = 0; j < T::FN; ++j) dmma_m8n8k4(acc[i][j][0], acc[i][j][1], af[i], bf[j]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty0 + 8u * s);
    }
    (void)ok;   // a wait that gave up has raised the CTA's abort flag

    // Epilogue: park the fragments as an image of the tile (rows contiguous) in the now idle
    // stage buffers, then all consumer threads walk it (see epilogue_common.cuh).
    consumer_barrier<T::CONSUMER_THREADS>();        // every consumer warp is done reading the stages
    if (*abort_flag) return;
    double *image = stage_base;
    constexpr int P = ImagePitch<T::BM>::value;
#pragma unroll
    for (int fi = 0; fi < T::FM; ++fi) {
        const int r = wm0 + fi * 8 + g;
#pragma unroll
        for (int fj = 0; fj < T::FN; ++fj) {
            if (T::CPLX) {
                const int c = (wn0w + fj * 8) / 2 + t;
                *reinterpret_cast<double2 *>(image + size_t(c * P + r) * 2) = make_double2(acc[fi][fj][0], acc[fi][fj][1]);
            } else {
                const int c = wn0w + fj * 8 + 2 * t;
                image[c * P + r] = acc[fi][fj][0];
                image[(c + 1) * P + r] = acc[fi][fj][1];
            }
        }
    }
    consumer_barrier<T::CONSUMER_THREADS>();
    if (p.cluster_split) {
        // the k slices of this tile are the CTAs of this cluster: add them up through distributed shared
        // memory, every CTA a share of the tile.  (Producer warps have returned; a CTA that gave up has
        // returned too and left the error word, which keeps D untouched as the two-kernel path does.)
        cluster_barrier();
        if (!(p.error_word && *static_cast<volatile int32_t *>(p.error_word) != 0))
            splitk_finish_cluster<double, W, T::BM, T::BN, T::CONSUMER_THREADS>(p, tc, image, rowD, colD, ctid);
        cluster_barrier();                              // nobody leaves while its image is being read
        return;
    }
    store_tile_image<double, W, T::BM, T::BN, T::CONSUMER_THREADS>(p, tc, image, rowD, colD, ctid);
}

}  // namespace btc

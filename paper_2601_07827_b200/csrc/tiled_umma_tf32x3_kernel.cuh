// fp32 contraction on the 5th-generation tensor cores (tcgen05.mma kind::tf32, accumulators in
// tensor memory), 3xTF32:  a*b = a_lo*b_hi + a_hi*b_lo + a_hi*b_hi  with x = x_hi + x_lo.
//
// CTA = 8 converter warps + 1 MMA warp, one CTA per SM, tile 128 x BN x 32 per stage.
//   converters  gather the strided A / B tiles through the offset tables with 16-byte global loads
//               into registers (the next stage's loads are in flight while the current stage is
//               converted), split every value into its TF32 head and tail, and store both as
//               separate operand tiles in the shared-memory layout the tensor core reads without
//               swizzling: 8 x 16-byte "core matrices".  An operand whose contiguous direction is
//               k is stored K-major, one whose contiguous direction is the free index MN-major;
//               the instruction descriptor carries that choice, so no transpose is ever made.
//   MMA warp    one elected lane waits for a stage ("full" mbarrier, 256 arrivals), issues the
//               4 k-steps x 3 MMAs of the stage and commits them to the stage's "empty" mbarrier;
//               after the last stage it commits to the accumulator barrier.
//   epilogue    the converter warps read the accumulator from tensor memory (each warp its own
//               32-lane quarter, one row of the tile per lane, so a warp's store of one column
//               is 32 consecutive rows of D) and apply alpha / beta through D's offset tables.
// Every wait is bounded; a wait that gives up raises the CTA abort flag and the error word, all
// roles fall through to the common tail, and the allocating warp always frees its tensor memory.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

template <int BN_, int STAGES_>
struct UmmaTile {
    static constexpr int BM = 128, BN = BN_, BK = 32;
    static constexpr int STAGES = STAGES_;
    static constexpr int CONVERTER_WARPS = 8, CONVERTER_THREADS = 256;
    static constexpr int THREADS = CONVERTER_THREADS + 32;          // + the MMA warp
    static constexpr int A_BYTES = BM * BK * 4, B_BYTES = BN * BK * 4;
    static constexpr int STAGE_BYTES = 2 * A_BYTES + 2 * B_BYTES;   // hi and lo tile of each operand
    static constexpr int TMEM_COLS = BN <= 32 ? 32 : BN <= 64 ? 64 : BN <= 128 ? 128 : 256;
    static constexpr int SLOTS_A = BM * BK / 4 / CONVERTER_THREADS; // 16-byte pieces per thread
    static constexpr int SLOTS_B = BN * BK / 4 / CONVERTER_THREADS;
    static_assert((BN * BK / 4) % CONVERTER_THREADS == 0, "B tile must divide among the converters");
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "BN must suit UMMA N and the epilogue split");
    // stages | row/col offsets | k offsets | full[S], empty[S], accum mbarriers | tmem ptr, abort
    static constexpr size_t SMEM_BYTES = size_t(STAGES) * STAGE_BYTES + size_t(2 * BM + 2 * BN + 2 * kKoffCap) * 8 +
                                         size_t(2 * STAGES + 1) * 8 + 16 + 1024;   // + slack to align the tiles
};

// ---- tcgen05 wrappers ---------------------------------------------------------------------------
__device__ __forceinline__ void tmem_alloc(unsigned smem_dst, int cols)
{
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish()
{
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, int cols)
{
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void umma_commit(unsigned bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void umma_tf32(unsigned tmem_c, uint64_t desc_a, uint64_t desc_b, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 ::"r"(tmem_c), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
                 : "memory");
}
__device__ __forceinline__ void tmem_load16(unsigned taddr, unsigned (&r)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                   "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                 : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_load_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ bool elect_one()
{
    unsigned pred = 0;
    asm volatile("{\n\t.reg .pred px;\n\telect.sync _|px, 0xffffffff;\n\tselp.u32 %0, 1, 0, px;\n\t}" : "=r"(pred)::"memory");
    return pred != 0;
}

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (all in 16-byte
// units), descriptor version 1, layout type (0: no swizzle, 1: 128-byte swizzle on 32-byte units).
__device__ __forceinline__ uint64_t umma_smem_desc(unsigned saddr, unsigned lbo_bytes, unsigned sbo_bytes, unsigned layout)
{
    return uint64_t((saddr >> 4) & 0x3fffu) | (uint64_t((lbo_bytes >> 4) & 0x3fffu) << 16) |
           (uint64_t((sbo_bytes >> 4) & 0x3fffu) << 32) | (uint64_t(1) << 46) | (uint64_t(layout & 7u) << 61);
}
// Instruction descriptor: fp32 accumulate, TF32 x TF32, M = 128, N, operand major-ness
__host__ __device__ constexpr unsigned umma_instr_desc(int n, bool a_mn_major, bool b_mn_major)
{
    return (1u << 4) | (2u << 7) | (2u << 10) | (unsigned(a_mn_major) << 15) | (unsigned(b_mn_major) << 16) |
           (unsigned(n >> 3) << 17) | (unsigned(128 >> 4) << 24);
}

// Byte position of a 16-byte piece inside one operand tile of R rows x 32 k.
//   k-contiguous operand, K-major, no swizzle: piece = 4 consecutive k of one row at
//        ((k/4) * R + row) * 16          [core matrix = 8 rows x 16 bytes; SBO 128, LBO 16 R]
//   free-index-contiguous operand, MN-major.  For 32-bit elements the tensor core accepts only
//   the 128-byte swizzle on 32-byte units here: atoms of 32 rows x 4 k (4 lines of 128 bytes,
//   the 32-byte unit of a line XORed with the line number), row atoms 512 bytes apart (LBO),
//   k atoms 16 R bytes apart (SBO); piece = 4 consecutive rows at one k.  Tiles are 1024-byte
//   aligned so that the XOR on address bits equals the XOR on tile offsets.
template <int R> __device__ __forceinline__ unsigned piece_kmajor(int row, int k) { return unsigned(((k >> 2) * R + row) * 16); }
template <int R> __device__ __forceinline__ unsigned piece_mnmajor(int row, int k)
{
    const int line = k & 3, unit = ((row & 31) >> 3) ^ line;
    return unsigned(((k >> 2) * (R / 32) + (row >> 5)) * 512 + line * 128 + unit * 32 + (row & 7) * 4);
}

struct F4 { float v[4]; };

// Which 16-byte piece converter slot s handles; the 8 lanes of a quarter warp store to 8
// different 16-byte bank groups.
//   dir 1 (k contiguous):    8 rows of one k-chunk, then the 8 chunks of the stage, then row groups
//   dir 0 (rows contiguous): 2 adjacent row pieces x 4 k of one atom line set, then 8-row groups,
//                            then the 8 k-atoms of the stage
template <int R> __device__ __forceinline__ void umma_slot(int s, int dir, int &row, int &k)
{
    if (dir == 1) {
        row = (s & 7) + 8 * (s >> 6);
        k = ((s >> 3) & 7) * 4;
    } else {
        const int rest = s >> 3;
        row = (rest % (R / 8)) * 8 + (s & 1) * 4;
        k = (rest / (R / 8)) * 4 + ((s >> 1) & 3);
    }
}

// One converter thread's pieces of an R x 32 operand tile: the global loads ...
template <int R, int SLOTS>
__device__ __forceinline__ void umma_gather(F4 (&reg)[SLOTS], const float *__restrict__ g, const int64_t *row_off,
                                            const int64_t *koff, int rows_valid, int64_t k0, int64_t k_end, int dir,
                                            int vec, int ctid)
{
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) {
        int row, k;
        umma_slot<R>(ctid + i * 256, dir, row, k);
#pragma unroll
        for (int e = 0; e < 4; ++e) reg[i].v[e] = 0.f;
        if (row < rows_valid && k0 + k < k_end) {
            if (vec == 4) {      // the 4 elements are 16 contiguous, aligned bytes and all in range
                const float4 x = *reinterpret_cast<const float4 *>(g + row_off[row] + koff[k0 + k]);
                reg[i].v[0] = x.x; reg[i].v[1] = x.y; reg[i].v[2] = x.z; reg[i].v[3] = x.w;
            } else if (dir == 1) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (k0 + k + e < k_end) reg[i].v[e] = g[row_off[row] + koff[k0 + k + e]];
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (row + e < rows_valid) reg[i].v[e] = g[row_off[row + e] + koff[k0 + k]];
            }
        }
    }
}

// ... and the split into TF32 head and tail with the stores into the hi / lo operand tiles
template <int R, int SLOTS>
__device__ __forceinline__ void umma_convert(const F4 (&reg)[SLOTS], unsigned hi_tile, unsigned lo_tile, int dir, int ctid)
{
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) {
        int row, k;
        umma_slot<R>(ctid + i * 256, dir, row, k);
        const unsigned pos = dir == 1 ? piece_kmajor<R>(row, k) : piece_mnmajor<R>(row, k);
        unsigned hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            hi[e] = __float_as_uint(reg[i].v[e]) & 0xffffe000u;
            lo[e] = __float_as_uint(reg[i].v[e] - __uint_as_float(hi[e])) & 0xffffe000u;
        }
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(hi_tile + pos), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(lo_tile + pos), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
    }
}

constexpr int kErrAccumWait = 3;

template <typename T>
__global__ void __launch_bounds__(T::THREADS, 1) tiled_umma_tf32x3_kernel(const TiledParams p)
{
    extern __shared__ __align__(16) unsigned char smem_unaligned[];
    // operand tiles must sit on 1024-byte boundaries of the shared-memory window (swizzled layouts)
    unsigned char *smem_raw = smem_unaligned +
        ((1024u - (static_cast<unsigned>(__cvta_generic_to_shared(smem_unaligned)) & 1023u)) & 1023u);
    int64_t *rowA = reinterpret_cast<int64_t *>(smem_raw + size_t(T::STAGES) * T::STAGE_BYTES);
    int64_t *rowD = rowA + T::BM;
    int64_t *colB = rowD + T::BM;
    int64_t *colD = colB + T::BN;
    int64_t *koffA = colD + T::BN;
    int64_t *koffB = koffA + kKoffCap;
    uint64_t *bars = reinterpret_cast<uint64_t *>(koffB + kKoffCap);      // full[S], empty[S], accum
    unsigned *tmem_slot = reinterpret_cast<unsigned *>(bars + 2 * T::STAGES + 1);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const unsigned smem0 = static_cast<unsigned>(__cvta_generic_to_shared(smem_raw));
    const unsigned full0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned empty0 = full0 + 8u * T::STAGES;
    const unsigned accum_bar = empty0 + 8u * T::STAGES;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const TileCoords tc = tile_coords<T::BM, T::BN, T::BK>(p);

    // ---- set-up: offset arrays, barriers, tensor memory ----
    {
        const int64_t hA = p.offA_h[tc.h], hB = p.offB_h[tc.h], hD = p.offD_h[tc.h];
        for (int i = tid; i < T::BM; i += T::THREADS) {
            const bool v = i < tc.rows_valid;
            rowA[i] = v ? p.offA_m[tc.m0 + i] + hA : 0;
            rowD[i] = v ? p.offD_m[tc.m0 + i] + hD : 0;
        }
        for (int i = tid; i < T::BN; i += T::THREADS) {
            const bool v = i < tc.cols_valid;
            colB[i] = v ? p.offB_n[tc.n0 + i] + hB : 0;
            colD[i] = v ? p.offD_n[tc.n0 + i] : 0;
        }
        const bool staged = tc.k_end - tc.k_begin <= kKoffCap;
        if (staged)
            for (int i = tid; i < int(tc.k_end - tc.k_begin); i += T::THREADS) {
                koffA[i] = p.offA_k[tc.k_begin + i];
                koffB[i] = p.offB_k[tc.k_begin + i];
            }
        if (tid == 0) {
            for (int s = 0; s < T::STAGES; ++s) {
                mbar_init(full0 + 8u * s, T::CONVERTER_THREADS);
                mbar_init(empty0 + 8u * s, 1);
            }
            mbar_init(accum_bar, 1);
            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (warp == T::CONVERTER_WARPS) {        // the MMA warp owns the tensor-memory allocation
            tmem_alloc(static_cast<unsigned>(__cvta_generic_to_shared(tmem_slot)), T::TMEM_COLS);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_acc = *tmem_slot;
    const bool staged = tc.k_end - tc.k_begin <= kKoffCap;
    const int64_t *ka = staged ? koffA - tc.k_begin : p.offA_k;
    const int64_t *kb = staged ? koffB - tc.k_begin : p.offB_k;

    if (warp < T::CONVERTER_WARPS) {
        // ------------------------------------------------------------- converters
        const float *gA = static_cast<const float *>(p.A), *gB = static_cast<const float *>(p.B);
        F4 ra[2][T::SLOTS_A], rb[2][T::SLOTS_B];
        if (tc.num_kt > 0) {
            umma_gather<T::BM, T::SLOTS_A>(ra[0], gA, rowA, ka, tc.rows_valid, tc.k_begin, tc.k_end, p.dirA, p.vecA, tid);
            umma_gather<T::BN, T::SLOTS_B>(rb[0], gB, colB, kb, tc.cols_valid, tc.k_begin, tc.k_end, p.dirB, p.vecB, tid);
        }
        bool ok = true;
#pragma unroll 1
        for (int kt2 = 0; ok && kt2 < tc.num_kt; kt2 += 2) {
#pragma unroll
            for (int par = 0; par < 2; ++par) {      // register buffers alternate with compile-time indices
                const int kt = kt2 + par;
                if (kt >= tc.num_kt) break;
                if (kt + 1 < tc.num_kt) {            // next stage's loads fly while this one is converted
                    const int64_t k1 = tc.k_begin + int64_t(kt + 1) * T::BK;
                    umma_gather<T::BM, T::SLOTS_A>(ra[par ^ 1], gA, rowA, ka, tc.rows_valid, k1, tc.k_end, p.dirA, p.vecA, tid);
                    umma_gather<T::BN, T::SLOTS_B>(rb[par ^ 1], gB, colB, kb, tc.cols_valid, k1, tc.k_end, p.dirB, p.vecB, tid);
                }
                const int s = kt % T::STAGES, round = kt / T::STAGES;
                if (round > 0 &&
                    !mbar_wait_bounded(empty0 + 8u * s, unsigned(round - 1) & 1u, abort_flag, p.error_word, kErrEmptyWait)) {
                    ok = false;
                    break;
                }
                const unsigned st = smem0 + unsigned(s) * T::STAGE_BYTES;
                umma_convert<T::BM, T::SLOTS_A>(ra[par], st, st + T::A_BYTES, p.dirA, tid);
                umma_convert<T::BN, T::SLOTS_B>(rb[par], st + 2 * T::A_BYTES, st + 2 * T::A_BYTES + T::B_BYTES, p.dirB, tid);
                proxy_fence_async();                 // the tensor core reads these stores through the async proxy
                mbar_arrive(full0 + 8u * s);
            }
        }

        // ------------------------------------------------------------- epilogue
        if (ok && mbar_wait_bounded(accum_bar, 0u, abort_flag, p.error_word, kErrAccumWait)) {
            tc_fence_after();
            float *D = static_cast<float *>(p.D);
            const float *C = static_cast<const float *>(p.C);
            const float alpha = float(p.alpha[0]), beta = float(p.beta[0]);
            const int quarter = warp & 3, half = warp >> 2;          // lanes 32 q .. 32 q + 31, column half
            const int row = quarter * 32 + lane;
            const bool row_ok = row < tc.rows_valid;
            const int64_t ro = rowD[row];
#pragma unroll 1
            for (int c0 = half * (T::BN / 2); c0 < (half + 1) * (T::BN / 2); c0 += 16) {
                unsigned r[16];
                tmem_load16(tmem_acc + (unsigned(quarter * 32) << 16) + unsigned(c0), r);
                tmem_load_wait();
                float cv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    cv[j] = (p.use_c && row_ok && c0 + j < tc.cols_valid) ? C[ro + colD[c0 + j]] : 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (row_ok && c0 + j < tc.cols_valid) {
                        float v = alpha * __uint_as_float(r[j]);
                        if (p.use_c) v += beta * cv[j];
                        D[ro + colD[c0 + j]] = v;
                    }
            }
            tc_fence_before();
        }
    } else {
        // ------------------------------------------------------------- MMA warp
        constexpr unsigned IDESC_KK = umma_instr_desc(T::BN, false, false);
        constexpr unsigned IDESC_MK = umma_instr_desc(T::BN, true, false);
        constexpr unsigned IDESC_KM = umma_instr_desc(T::BN, false, true);
        constexpr unsigned IDESC_MM = umma_instr_desc(T::BN, true, true);
        const bool a_mn = p.dirA == 0, b_mn = p.dirB == 0;
        const unsigned idesc = a_mn ? (b_mn ? IDESC_MM : IDESC_MK) : (b_mn ? IDESC_KM : IDESC_KK);
        // per operand: layout type, leading / stride byte offsets, start advance of one k-step (8 k)
        const unsigned a_lay = a_mn ? 1u : 0u, a_lbo = a_mn ? 512u : 16u * T::BM, a_sbo = a_mn ? 16u * T::BM : 128u;
        const unsigned b_lay = b_mn ? 1u : 0u, b_lbo = b_mn ? 512u : 16u * T::BN, b_sbo = b_mn ? 16u * T::BN : 128u;
        const unsigned a_step = 32u * T::BM, b_step = 32u * T::BN;   // two k-chunks, or two k-atoms
        const bool leader = elect_one();
        bool ok = true;
#pragma unroll 1
        for (int kt = 0; ok && kt < tc.num_kt; ++kt) {
            const int s = kt % T::STAGES, round = kt / T::STAGES;
            if (!mbar_wait_bounded(full0 + 8u * s, unsigned(round) & 1u, abort_flag, p.error_word, kErrFullWait)) {
                ok = false;
                break;
            }
            tc_fence_after();
            if (leader) {
                const unsigned st = smem0 + unsigned(s) * T::STAGE_BYTES;
                const unsigned a_hi = st, a_lo = st + T::A_BYTES, b_hi = st + 2 * T::A_BYTES, b_lo = b_hi + T::B_BYTES;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint64_t dah = umma_smem_desc(a_hi + j * a_step, a_lbo, a_sbo, a_lay);
                    const uint64_t dal = umma_smem_desc(a_lo + j * a_step, a_lbo, a_sbo, a_lay);
                    const uint64_t dbh = umma_smem_desc(b_hi + j * b_step, b_lbo, b_sbo, b_lay);
                    const uint64_t dbl = umma_smem_desc(b_lo + j * b_step, b_lbo, b_sbo, b_lay);
                    umma_tf32(tmem_acc, dal, dbh, idesc, (kt > 0 || j > 0) ? 1u : 0u);
                    umma_tf32(tmem_acc, dah, dbl, idesc, 1u);
                    umma_tf32(tmem_acc, dah, dbh, idesc, 1u);
                }
                umma_commit(empty0 + 8u * s);        // fires when these MMAs have read the stage
                if (kt + 1 == tc.num_kt) umma_commit(accum_bar);
            }
            __syncwarp();
        }
        tc_fence_before();
    }

    // ---- common tail: every role arrives here, also after an abort ----
    __syncthreads();
    if (warp == T::CONVERTER_WARPS) {
        tc_fence_after();
        tmem_dealloc(tmem_acc, T::TMEM_COLS);
    }
}

}  // namespace btc

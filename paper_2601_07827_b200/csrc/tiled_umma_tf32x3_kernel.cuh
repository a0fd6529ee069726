// fp32 contraction on the 5th-generation tensor cores (tcgen05.mma kind::tf32, accumulators in
// tensor memory), 3xTF32:  a*b = a_lo*b_hi + a_hi*b_lo + a_hi*b_hi  with x = x_hi + x_lo.
//
// CTA = 8 converter warps + 1 MMA warp, one CTA per SM, tile 128 x BN x 32 per stage.
//   converters  gather the strided A / B tiles through the offset tables with 16-byte global loads
//               into registers (the next stage's loads are in flight while the current stage is
//               converted), split every value into its TF32 head and tail, and store both as
//               separate operand tiles in the swizzled shared-memory layouts the tensor core
//               reads (a warp's load covers whole 128-byte lines of global memory and its stores
//               are free of bank conflicts).  An operand whose contiguous direction is
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

template <int BN_, int STAGES_, int PREFETCH_ = 2>
struct UmmaTile {
    static constexpr int BM = 128, BN = BN_, BK = 32;
    static constexpr int PREFETCH = PREFETCH_;                       // stages of global loads in flight per thread
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
// units), descriptor version 1, layout type (1: 128-byte swizzle on 32-byte units, 2: 128-byte swizzle on 16-byte units).
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

// Byte position of a 16-byte piece inside one operand tile of R rows x 32 k.  Both layouts are
// 128-byte swizzles, and tiles are 1024-byte aligned so that the XOR on address bits equals the
// XOR on tile offsets.
//   k-contiguous operand, K-major, 128-byte swizzle on 16-byte units: a row is its 32 k = 128
//        bytes, 8 rows form a 1024-byte atom (SBO 1024), and the 16-byte chunk index of a row is
//        XORed with (row mod 8); piece = 4 consecutive k of one row.  A k-step of 8 advances the
//        start address by 32 bytes inside the atom.
//   free-index-contiguous operand, MN-major.  For 32-bit elements the tensor core accepts only
//        the 128-byte swizzle on 32-byte units here: atoms of 32 rows x 4 k (4 lines of 128
//        bytes, the 32-byte unit of a line XORed with the line number), row atoms 512 bytes
//        apart (LBO), k atoms 16 R bytes apart (SBO); piece = 4 consecutive rows at one k.
template <int R> __device__ __forceinline__ unsigned piece_kmajor(int row, int k)
{
    return unsigned((row >> 3) * 1024 + (row & 7) * 128 + ((((k >> 2) ^ row) & 7) << 4));
}
template <int R> __device__ __forceinline__ unsigned piece_mnmajor(int row, int k)
{
    const int line = k & 3, unit = ((row & 31) >> 3) ^ line;
    return unsigned(((k >> 2) * (R / 32) + (row >> 5)) * 512 + line * 128 + unit * 32 + (row & 7) * 4);
}

struct F4 { float v[4]; };

// What a converter thread needs to address one operand: the tile's row offsets (shared memory),
// the k offsets indexed by absolute k (the staged copy in shared memory, or the global table),
// and the valid ranges.
struct UmmaOperand {
    const float *g;
    const int64_t *row_off;
    const int64_t *koff;
    int rows_valid;
    int64_t k_begin, k_end;
    int dir;                     // 1: k is the contiguous direction, 0: the rows are
};

// The 16-byte pieces of an R x 32 operand tile that converter thread ctid handles: R / 32 slots,
// slot i = 4 consecutive elements along the contiguous direction starting at (row r0 + 32 i, k kq).
//   dir 1 (k contiguous):    r0 = ctid / 8, kq = 4 (ctid mod 8): 8 lanes read the 128 bytes of a row
//   dir 0 (rows contiguous): r0 = 4 (ctid mod 8), kq = ctid / 8: 8 lanes read 32 rows of one k
// Either way a warp's global load covers 4 whole 128-byte lines, the 8 lanes of a quarter warp
// store to 8 different 16-byte bank groups, a thread's slots share their k (one k-offset look-up
// per stage) and keep their rows (row offsets and shared-memory positions are loop invariants:
// slot i lies i * pstep bytes behind slot 0 in both layouts).
template <int SLOTS> struct UmmaLane {
    const float *base[SLOTS];    // vector path: operand base + row offset of slot i (slot 0 of the tile if outside)
    unsigned pos0, pstep;
    unsigned rows_in;            // vector path: bit i = slot i lies inside the tile's rows
    int r0, kq;
};

template <int R, int SLOTS, bool VEC>
__device__ __forceinline__ void umma_lane_init(UmmaLane<SLOTS> &l, const UmmaOperand &o, int ctid)
{
    l.r0 = o.dir == 1 ? ctid >> 3 : (ctid & 7) * 4;
    l.kq = o.dir == 1 ? (ctid & 7) * 4 : ctid >> 3;
    l.pos0 = o.dir == 1 ? piece_kmajor<R>(l.r0, l.kq) : piece_mnmajor<R>(l.r0, l.kq);
    l.pstep = o.dir == 1 ? 4096u : 512u;
    l.rows_in = 0;
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) {
        const bool in = l.r0 + 32 * i < o.rows_valid;
        l.rows_in |= unsigned(in) << i;
        l.base[i] = VEC ? o.g + o.row_off[in ? l.r0 + 32 * i : 0] : o.g;
    }
}

// The global loads of one stage ...  They carry no predicate and sit under no branch: a piece
// outside the tile reads a valid element of the tile instead and is zeroed when it is converted.
// A conditional load would end in a select that waits for the data, one memory round trip per
// piece; this way the loads of a stage are issued back to back.  VEC: every piece is 16
// contiguous, aligned bytes that are in range together; otherwise its 4 elements are loaded one
// by one through the tables.
template <int SLOTS, bool VEC>
__device__ __forceinline__ void umma_gather(F4 (&reg)[SLOTS], const UmmaLane<SLOTS> &l, const UmmaOperand &o, int64_t k0)
{
    if (VEC) {
        const int64_t kofs = o.koff[k0 + l.kq < o.k_end ? k0 + l.kq : o.k_begin];
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) {
            const float4 x = *reinterpret_cast<const float4 *>(l.base[i] + kofs);
            reg[i].v[0] = x.x, reg[i].v[1] = x.y, reg[i].v[2] = x.z, reg[i].v[3] = x.w;
        }
    } else {
#pragma unroll
        for (int i = 0; i < SLOTS; ++i)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int re = l.r0 + 32 * i + (o.dir == 1 ? 0 : e);
                const int64_t ke = k0 + l.kq + (o.dir == 1 ? e : 0);
                const bool in = re < o.rows_valid && ke < o.k_end;
                reg[i].v[e] = o.g[o.row_off[in ? re : 0] + o.koff[in ? ke : o.k_begin]];
            }
    }
}

// ... and the split into TF32 head and tail with the stores into the hi / lo operand tiles.
// `full`: the whole R x 32 stage lies inside the tensor, nothing has to be zeroed.
template <int SLOTS>
__device__ __forceinline__ void umma_convert(const F4 (&reg)[SLOTS], const UmmaLane<SLOTS> &l, const UmmaOperand &o,
                                             int64_t k0, unsigned hi_tile, unsigned lo_tile, bool full)
{
#pragma unroll
    for (int i = 0; i < SLOTS; ++i) {
        unsigned hi[4], lo[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            float x = reg[i].v[e];
            if (!full) {
                const int re = l.r0 + 32 * i + (o.dir == 1 ? 0 : e);
                const int64_t ke = k0 + l.kq + (o.dir == 1 ? e : 0);
                if (re >= o.rows_valid || ke >= o.k_end) x = 0.f;
            }
            hi[e] = __float_as_uint(x) & 0xffffe000u;
            lo[e] = __float_as_uint(x - __uint_as_float(hi[e])) & 0xffffe000u;
        }
        const unsigned pos = l.pos0 + unsigned(i) * l.pstep;
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(hi_tile + pos), "r"(hi[0]), "r"(hi[1]), "r"(hi[2]), "r"(hi[3]) : "memory");
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(lo_tile + pos), "r"(lo[0]), "r"(lo[1]), "r"(lo[2]), "r"(lo[3]) : "memory");
    }
}

constexpr int kErrAccumWait = 3;

// Debug builds (-DBTC_STAMPS) add up the SM clock cycles one thread spends in each phase.
#ifdef BTC_STAMPS
#define BTC_PHASE_BEGIN() long long phase_t0 = clock64()
#define BTC_PHASE_END(acc) do { const long long phase_t1 = clock64(); (acc) += phase_t1 - phase_t0; phase_t0 = phase_t1; } while (0)
#define BTC_PHASE_STORE(p, who, slot, acc) do { if ((who) && (p).stamps && blockIdx.x < 512) (p).stamps[blockIdx.x * 8 + (slot)] = (acc); } while (0)
#else
#define BTC_PHASE_BEGIN() do { } while (0)
#define BTC_PHASE_END(acc) do { } while (0)
#define BTC_PHASE_STORE(p, who, slot, acc) do { } while (0)
#endif

// The converter warps' main loop.  A register ring keeps the loads of the next PF stages in
// flight while a stage is converted; ring positions are compile-time register indices.
template <typename T, bool VEC>
__device__ __forceinline__ bool umma_converter_loop(const TiledParams &p, const TileCoords &tc, const UmmaOperand &opA,
                                                    const UmmaOperand &opB, unsigned smem0, unsigned full0, unsigned empty0,
                                                    volatile int *abort_flag, int tid)
{
    constexpr int PF = T::PREFETCH, NB = PF + 1;
    F4 ra[NB][T::SLOTS_A], rb[NB][T::SLOTS_B];
    UmmaLane<T::SLOTS_A> la;
    UmmaLane<T::SLOTS_B> lb;
    umma_lane_init<T::BM, T::SLOTS_A, VEC>(la, opA, tid);
    umma_lane_init<T::BN, T::SLOTS_B, VEC>(lb, opB, tid);
    const bool rows_full = opA.rows_valid == T::BM && opB.rows_valid == T::BN;
#pragma unroll
    for (int q = 0; q < PF; ++q)
        if (q < tc.num_kt) {
            const int64_t kq = tc.k_begin + int64_t(q) * T::BK;
            umma_gather<T::SLOTS_A, VEC>(ra[q], la, opA, kq);
            umma_gather<T::SLOTS_B, VEC>(rb[q], lb, opB, kq);
        }
    bool ok = true;
    long long t_gather = 0, t_wait = 0, t_convert = 0, t_signal = 0;
    (void)t_gather; (void)t_wait; (void)t_convert; (void)t_signal;
    BTC_PHASE_BEGIN();
#pragma unroll 1
    for (int kt0 = 0; ok && kt0 < tc.num_kt; kt0 += NB) {
#pragma unroll
        for (int b = 0; b < NB; ++b) {
            const int kt = kt0 + b;
            if (kt >= tc.num_kt) break;
            const int64_t k0 = tc.k_begin + int64_t(kt) * T::BK;
            if (kt + PF < tc.num_kt) {
                const int64_t k1 = k0 + int64_t(PF) * T::BK;
                umma_gather<T::SLOTS_A, VEC>(ra[(b + PF) % NB], la, opA, k1);
                umma_gather<T::SLOTS_B, VEC>(rb[(b + PF) % NB], lb, opB, k1);
            }
            BTC_PHASE_END(t_gather);
            const int s = kt % T::STAGES, round = kt / T::STAGES;
            if (round > 0 &&
                !mbar_wait_bounded(empty0 + 8u * s, unsigned(round - 1) & 1u, abort_flag, p.error_word, kErrEmptyWait)) {
                ok = false;
                break;
            }
            BTC_PHASE_END(t_wait);
            const unsigned st = smem0 + unsigned(s) * T::STAGE_BYTES;
            const bool full = rows_full && k0 + T::BK <= tc.k_end;
            umma_convert<T::SLOTS_A>(ra[b], la, opA, k0, st, st + T::A_BYTES, full);
            umma_convert<T::SLOTS_B>(rb[b], lb, opB, k0, st + 2 * T::A_BYTES, st + 2 * T::A_BYTES + T::B_BYTES, full);
            BTC_PHASE_END(t_convert);
            proxy_fence_async();                 // the tensor core reads these stores through the async proxy
            mbar_arrive(full0 + 8u * s);
            BTC_PHASE_END(t_signal);
        }
    }
    BTC_PHASE_STORE(p, tid == 0, 0, t_gather);
    BTC_PHASE_STORE(p, tid == 0, 1, t_wait);
    BTC_PHASE_STORE(p, tid == 0, 2, t_convert);
    BTC_PHASE_STORE(p, tid == 0, 3, t_signal);
    return ok;
}

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

    if (warp < T::CONVERTER_WARPS) {
        // ------------------------------------------------------------- converters
        const UmmaOperand opA = {static_cast<const float *>(p.A), rowA, staged ? koffA - tc.k_begin : p.offA_k,
                                 tc.rows_valid, tc.k_begin, tc.k_end, p.dirA};
        const UmmaOperand opB = {static_cast<const float *>(p.B), colB, staged ? koffB - tc.k_begin : p.offB_k,
                                 tc.cols_valid, tc.k_begin, tc.k_end, p.dirB};
        const bool ok = (p.vecA == 4 && p.vecB == 4)
                            ? umma_converter_loop<T, true>(p, tc, opA, opB, smem0, full0, empty0, abort_flag, tid)
                            : umma_converter_loop<T, false>(p, tc, opA, opB, smem0, full0, empty0, abort_flag, tid);

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
        const unsigned a_lay = a_mn ? 1u : 2u, a_lbo = a_mn ? 512u : 16u, a_sbo = a_mn ? 16u * T::BM : 1024u;
        const unsigned b_lay = b_mn ? 1u : 2u, b_lbo = b_mn ? 512u : 16u, b_sbo = b_mn ? 16u * T::BN : 1024u;
        const unsigned a_step = a_mn ? 32u * T::BM : 32u, b_step = b_mn ? 32u * T::BN : 32u;   // two k-atoms, or 8 k of a row
        const bool leader = elect_one();
        bool ok = true;
        long long t_full = 0, t_issue = 0;
        (void)t_full; (void)t_issue;
        BTC_PHASE_BEGIN();
#pragma unroll 1
        for (int kt = 0; ok && kt < tc.num_kt; ++kt) {
            const int s = kt % T::STAGES, round = kt / T::STAGES;
            if (!mbar_wait_bounded(full0 + 8u * s, unsigned(round) & 1u, abort_flag, p.error_word, kErrFullWait)) {
                ok = false;
                break;
            }
            BTC_PHASE_END(t_full);
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
            BTC_PHASE_END(t_issue);
        }
        BTC_PHASE_STORE(p, lane == 0, 4, t_full);
        BTC_PHASE_STORE(p, lane == 0, 5, t_issue);
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

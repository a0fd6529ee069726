// fp32 contraction on the 5th-generation tensor cores (tcgen05.mma kind::tf32, accumulators in
// tensor memory), 3xTF32:  a*b = a_lo*b_hi + a_hi*b_lo + a_hi*b_hi  with x = x_hi + x_lo.
//
// Persistent CTAs (one per SM) of 4 epilogue + 4 converter + 4 producer warps + 1 MMA warp walk the
// list of 128 x BN tiles, 32 k per stage.  Shared memory holds a deep ring of "raw" stages and a
// short ring of "tail" stages, tensor memory two accumulators.
//   producers   gather the strided A / B tiles through the offset tables with asynchronous
//               16-byte copies (zero-filled outside the tensor) straight into the swizzled
//               operand layouts the tensor core reads.  Asynchronous copies keep far more bytes
//               in flight per SM than loads into registers can, which is what bounds this kernel.
//               An operand whose contiguous direction is k is stored K-major, one whose
//               contiguous direction is the free index MN-major; the instruction descriptor
//               carries that choice, so no transpose is ever made.
//   converters  The tensor core reads only the upper 19 bits of a 32-bit operand element, so the
//               raw fp32 stage already is the head operand x_hi.  The converters read it, form
//               the tail x - x_hi (exact in fp32) and store it at the same position of a tail
//               stage: a position-independent, conflict-free pass over the stage.
//   MMA warp    one elected lane waits for a tail stage ("tail full"; it implies the raw stage),
//               issues the 4 k-steps x 3 MMAs and commits them to the "raw empty" and "tail
//               empty" mbarriers; after a tile's last stage it commits to that accumulator's
//               "full" barrier and moves on to the other accumulator.
//   epilogue    warp w reads lanes 32 w .. 32 w + 31 of the finished accumulator (one row of the
//               tile per lane, so a warp's store of one column is 32 consecutive rows of D),
//               applies alpha / beta through D's offset tables and releases the accumulator,
//               while the other roles already work on the next tile.
// A_TMA variants: when every (tile, stage) of the M-side operand is a rectangular box of a tensor
// of at most five dimensions, one producer thread fetches it with a single bulk tensor copy
// (cp.async.bulk.tensor, completion counted in bytes on the stage's "raw full" mbarrier) instead of
// 128 threads issuing 16-byte copies; the box lands row by row (k contiguous) or column by column
// (rows contiguous) and the converters move it on to tensor memory.  The N side keeps its gather.
// Every wait is bounded; a wait that gives up raises the CTA abort flag and the error word, all
// roles fall through to the common tail, and the allocating warp always frees its tensor memory.
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

template <int BN_, int RAW_STAGES_, int TAIL_STAGES_, bool A_TMEM_ = false, int CONVERTER_GROUPS_ = 1, int BK_ = 32, bool A_TMA_ = false,
          int SUBS_ = 1>
struct UmmaTile {
    static constexpr int BM = 128, BN = BN_, BK = BK_;
    static constexpr int KSTEPS = BK_ / 8;                           // tensor-core instructions of K = 8 per sub-stage
    // A stage (the unit the roles hand to one another through mbarriers) holds SUBS sub-stages of BK
    // k each, laid out one after the other.  A hand-off costs several hundred cycles whatever the
    // stage holds, so two sub-stages per stage halve that cost per k.
    static constexpr int SUBS = SUBS_;
    static constexpr int RAW_STAGES = RAW_STAGES_, TAIL_STAGES = TAIL_STAGES_;
    // A_TMA: the M-side tile of a stage arrives by one bulk tensor copy (needs A_TMEM: the box is
    // not in a layout the tensor core reads, the converters take it to tensor memory)
    static constexpr bool A_TMA = A_TMA_;
    static_assert(BK_ == 32 || (BK_ == 24 && A_TMA_), "stages of 24 exist for the bulk-copy variants only");
    static_assert(!A_TMA_ || A_TMEM_, "the bulk-copy variants pass the M side through tensor memory");
    // A_TMEM: the M-side operand reaches the tensor core through tensor memory (the converters
    // write its head and tail there), so the tensor core reads only the N-side operand from
    // shared memory and a tail stage holds only that operand's tail
    static constexpr bool A_TMEM = A_TMEM_;
    static constexpr int EPILOGUE_WARPS = 4, EPILOGUE_THREADS = 128;  // warps 0-3: one tensor-memory lane quarter each
    // converter groups of 4 warps (128 threads = the tile's 128 rows) take the stages in turn
    static constexpr int CONVERTER_GROUPS = CONVERTER_GROUPS_;
    static constexpr int CONVERTER_WARPS = 4 * CONVERTER_GROUPS_, CONVERTER_THREADS = 128;   // threads per group
    static constexpr int PRODUCER_WARPS = 4, PRODUCER_THREADS = 128;
    static constexpr int MMA_WARP = EPILOGUE_WARPS + CONVERTER_WARPS + PRODUCER_WARPS;
    static constexpr int THREADS = 32 * (MMA_WARP + 1);
    // a k-contiguous N-side tile keeps 128-byte rows whatever BK is (the swizzle atom)
    static constexpr int A_BYTES = BM * BK * 4, B_BYTES = BN * 32 * 4;
    static constexpr int SUB_BYTES = A_BYTES + B_BYTES;             // one sub-stage of a raw stage: M-side tile, N-side tile
    static constexpr int STAGE_BYTES = SUBS_ * SUB_BYTES;           // a raw stage
    static_assert(A_BYTES % 1024 == 0, "operand tiles sit on 1024-byte boundaries");
    static constexpr int TAIL_SUB_BYTES = A_TMEM_ ? B_BYTES : SUB_BYTES;
    static constexpr int TAIL_BYTES = SUBS_ * TAIL_SUB_BYTES;
    static constexpr int TAIL_B_OFFSET = A_TMEM_ ? 0 : A_BYTES;     // where the N-side tail sits in a tail stage
    static constexpr int ACC_COLS = BN <= 32 ? 32 : BN <= 64 ? 64 : BN <= 128 ? 128 : 256;   // one accumulator
    static constexpr int A_SUB_COLS = A_TMEM_ ? 2 * BK : 0;         // head + tail of one sub-stage of the M-side operand
    static constexpr int A_COLS = SUBS_ * A_SUB_COLS;
    static constexpr int TMEM_USED = 2 * ACC_COLS + TAIL_STAGES_ * A_COLS;
    static constexpr int TMEM_COLS = TMEM_USED <= 32 ? 32 : TMEM_USED <= 64 ? 64 : TMEM_USED <= 128 ? 128 : TMEM_USED <= 256 ? 256 : 512;
    static_assert(TMEM_USED <= 512, "accumulators and operand stages must fit the 512 tensor-memory columns");
    // 16-byte pieces per converter thread in the position-independent pass (whole stage, or its N side)
    static constexpr int PIECES = (A_TMEM_ ? B_BYTES : SUB_BYTES) / 16 / CONVERTER_THREADS;
    static constexpr int NUM_BARS = 2 * RAW_STAGES + 2 * TAIL_STAGES + 9;    // ... + the drain barrier of the abort path
    static_assert(B_BYTES % (16 * CONVERTER_THREADS) == 0, "a stage must divide among the converters");
    static_assert(BN % 32 == 0 && BN >= 32 && BN <= 256, "BN must suit UMMA N and the epilogue split");
    // stages | row/col offsets | k offsets | mbarriers | tmem ptr, abort
    static constexpr size_t SMEM_BYTES = size_t(RAW_STAGES) * STAGE_BYTES + size_t(TAIL_STAGES) * TAIL_BYTES +
                                         size_t(2 * BM + 4 * BN + 2 * kKoffCap) * 8 + size_t(NUM_BARS) * 8 + 16 +
                                         1024;   // + slack to align the tiles
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
// same with the M-side operand read from tensor memory (lane = row, one column per k)
__device__ __forceinline__ void umma_tf32_ts(unsigned tmem_c, unsigned tmem_a, uint64_t desc_b, unsigned idesc, unsigned accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, {%5, %6, %7, %8}, p;\n\t}"
                 ::"r"(tmem_c), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate), "r"(0u), "r"(0u), "r"(0u), "r"(0u)
                 : "memory");
}
// 32 consecutive columns of this lane's tensor-memory row
__device__ __forceinline__ void tmem_store32(unsigned taddr, const float (&v)[32])
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
                 "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
                 ::"r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]),
                   "f"(v[8]), "f"(v[9]), "f"(v[10]), "f"(v[11]), "f"(v[12]), "f"(v[13]), "f"(v[14]), "f"(v[15]),
                   "f"(v[16]), "f"(v[17]), "f"(v[18]), "f"(v[19]), "f"(v[20]), "f"(v[21]), "f"(v[22]), "f"(v[23]),
                   "f"(v[24]), "f"(v[25]), "f"(v[26]), "f"(v[27]), "f"(v[28]), "f"(v[29]), "f"(v[30]), "f"(v[31])
                 : "memory");
}
// 8 consecutive columns of this lane's tensor-memory row
__device__ __forceinline__ void tmem_store8(unsigned taddr, const float *v)
{
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 ::"r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7])
                 : "memory");
}
__device__ __forceinline__ void tmem_store_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// one arrival on the barrier plus `bytes` that a bulk copy will report on it
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bulk tensor copy of one box (five coordinates, dimension 0 first) into shared memory; its bytes
// are reported on `bar`.  Dimension 0's coordinate must be a multiple of four elements.
__device__ __forceinline__ void tma_load_box(unsigned dst, const CUtensorMap *map, unsigned bar, int c0, int c1, int c2, int c3, int c4)
{
    asm volatile("cp.async.bulk.tensor.5d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(c4), "r"(bar) : "memory");
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


// What a producer thread needs to address one operand: the tile's row offsets (shared memory),
// the k offsets indexed by absolute k (the staged copy in shared memory, or the global table),
// and the valid ranges.
struct UmmaOperand {
    const float *g;
    const int64_t *row_off;
    const int64_t *koff;
    int rows_valid;
    int64_t k_begin, k_end;
    int dir;                     // 1: k is the contiguous direction, 0: the rows are
    int vec;                     // 4: every 16-byte piece is contiguous, aligned and in range as a whole
    const OffsetSpans *spans;    // debug builds: what the offsets are checked against
    int which;
};

// The 16-byte pieces of an R x 32 operand tile that producer thread pt (0..127) copies: R / 16
// slots, each 4 consecutive elements along the contiguous direction.
//   dir 1 (k contiguous):    rows r0 + 16 i at k kq,  r0 = pt / 8, kq = 4 (pt mod 8):
//                            8 lanes copy the 128 bytes of one row
//   dir 0 (rows contiguous): rows r0 + 32 j at k kq + 16 h,  r0 = 4 (pt mod 8), kq = pt / 8,
//                            slot i = j + (R / 32) h: 8 lanes copy 32 rows of one k
// Either way a warp's copy covers 4 whole 128-byte lines of global memory, a thread keeps its
// rows for the whole k loop (row offsets and shared-memory positions are loop invariants) and
// needs at most two k-offset look-ups per stage.
template <int R> struct UmmaProducerLane {
    static constexpr int SLOTS = R / 16;
    int64_t rowoff[SLOTS];       // element offset of slot i's first row (0 if outside the tile)
    unsigned rows_in;            // bit i = slot i's first row lies inside the tile
    unsigned pos0;               // byte position of slot 0 in the operand tile
    int r0, kq;
};

template <int R> __device__ __forceinline__ int umma_slot_row(int dir, int r0, int i) { return dir == 1 ? r0 + 16 * i : r0 + 32 * (i % (R / 32)); }
template <int R> __device__ __forceinline__ int umma_slot_half(int dir, int i) { return dir == 1 ? 0 : i / (R / 32); }
template <int R> __device__ __forceinline__ unsigned umma_slot_pos(int dir, int i)
{
    return dir == 1 ? 2048u * unsigned(i) : 512u * unsigned(i % (R / 32)) + unsigned(R * 64) * unsigned(i / (R / 32));
}

template <int R>
__device__ __forceinline__ void umma_producer_init(UmmaProducerLane<R> &l, const UmmaOperand &o, int pt)
{
    l.r0 = o.dir == 1 ? pt >> 3 : (pt & 7) * 4;
    l.kq = o.dir == 1 ? (pt & 7) * 4 : pt >> 3;
    l.pos0 = o.dir == 1 ? piece_kmajor<R>(l.r0, l.kq) : piece_mnmajor<R>(l.r0, l.kq);
    l.rows_in = 0;
#pragma unroll
    for (int i = 0; i < UmmaProducerLane<R>::SLOTS; ++i) {
        const int row = umma_slot_row<R>(o.dir, l.r0, i);
        const bool in = row < o.rows_valid;
        l.rows_in |= unsigned(in) << i;
        l.rowoff[i] = o.row_off[in ? row : 0];
    }
}

// The k offsets a producer thread needs for one stage (vector path): at most two look-ups.
struct UmmaStageOffsets {
    int64_t kofs0, kofs1;
    bool in0, in1;
};
template <int R, int BK = 32>
__device__ __forceinline__ UmmaStageOffsets umma_lookup(const UmmaProducerLane<R> &l, const UmmaOperand &o, int64_t k0)
{
    UmmaStageOffsets s;
    const int64_t ka = k0 + l.kq, kb = ka + 16;
    s.in0 = ka < o.k_end && (BK == 32 || l.kq < BK);
    s.in1 = o.dir == 0 && kb < o.k_end && l.kq + 16 < BK;
    s.kofs0 = o.koff[s.in0 ? ka : o.k_begin];
    s.kofs1 = o.koff[s.in1 ? kb : o.k_begin];
    return s;
}

// The copies of one operand for one stage.  Look-ups first, copies after: a copy is an ordered
// memory operation, so a look-up placed behind one would wait for it; the caller therefore looks
// up a stage's offsets (`so`, vector path) before it issues the copies of the stage before.
// A stage holds BK <= 32 k: slots whose k lies beyond BK are skipped (their place in the tile is
// never read by the tensor core).
template <int R, int BK = 32>
__device__ __forceinline__ void umma_produce(unsigned tile, const UmmaProducerLane<R> &l, const UmmaOperand &o, int64_t k0,
                                             const UmmaStageOffsets &so)
{
    constexpr int SLOTS = UmmaProducerLane<R>::SLOTS;
    if (BK < 32 && l.kq >= BK) return;
    if (o.vec == 4) {
#pragma unroll
        for (int i = 0; i < SLOTS; ++i) {
            const bool second = umma_slot_half<R>(o.dir, i) != 0;
            if (BK < 32 && second && l.kq + 16 >= BK) continue;
            bool valid = ((l.rows_in >> i) & 1u) && (second ? so.in1 : so.in0);
            int64_t off = l.rowoff[i] + (second ? so.kofs1 : so.kofs0);
            if (valid && !BTC_IN_SPAN(*o.spans, o.which, off, 4)) { valid = false; off = 0; }
            cp_async_bytes<16>(tile + l.pos0 + umma_slot_pos<R>(o.dir, i), o.g + off, valid);
        }
    } else {
#pragma unroll 2
        for (int i = 0; i < SLOTS; ++i) {
            const int row = umma_slot_row<R>(o.dir, l.r0, i);
            if (BK < 32 && l.kq + 16 * umma_slot_half<R>(o.dir, i) >= BK) continue;
            const int64_t k = k0 + l.kq + 16 * umma_slot_half<R>(o.dir, i);
            int64_t off[4];
            bool in[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int re = row + (o.dir == 1 ? 0 : e);
                const int64_t ke = k + (o.dir == 1 ? e : 0);
                in[e] = re < o.rows_valid && ke < o.k_end;
                off[e] = in[e] ? o.row_off[re] + o.koff[ke] : 0;
                if (in[e] && !BTC_IN_SPAN(*o.spans, o.which, off[e], 1)) { in[e] = false; off[e] = 0; }
            }
#pragma unroll
            for (int e = 0; e < 4; ++e)
                cp_async_bytes<4>(tile + l.pos0 + umma_slot_pos<R>(o.dir, i) + 4u * e, o.g + off[e], in[e]);
        }
    }
}

constexpr int kErrAccumWait = 3, kErrTailFullWait = 4, kErrTailEmptyWait = 5, kErrGroupSync = 6;


// Group-wide rendezvous on an mbarrier (every member arrives, then waits with a bound): unlike a
// named barrier it cannot hang when a member has left after an abort.
__device__ __forceinline__ bool umma_group_sync(unsigned bar, unsigned parity, volatile int *abort_flag, int *error_word,
                                                unsigned poll_limit = kWaitPollLimit)
{
    mbar_arrive(bar);
    return mbar_wait_bounded(bar, parity, abort_flag, error_word, kErrGroupSync, poll_limit);
}

// Persistent: CTA b works on the items b, b + gridDim.x, ... of the (tile, batch) list; all roles
// walk that list with the same counters.  Tensor memory holds two accumulators, so the epilogue
// of one tile overlaps the main loop of the next; the shared-memory rings run across tiles.
template <typename T>
__global__ void __launch_bounds__(T::THREADS, 1) tiled_umma_tf32x3_kernel(const TiledParams p, const __grid_constant__ CUtensorMap tmapA)
{
    extern __shared__ __align__(16) unsigned char smem_unaligned[];
    // operand tiles must sit on 1024-byte boundaries of the shared-memory window (swizzled layouts)
    unsigned char *smem_raw = smem_unaligned +
        ((1024u - (static_cast<unsigned>(__cvta_generic_to_shared(smem_unaligned)) & 1023u)) & 1023u);
    int64_t *rowA = reinterpret_cast<int64_t *>(smem_raw + size_t(T::RAW_STAGES) * T::STAGE_BYTES + size_t(T::TAIL_STAGES) * T::TAIL_BYTES);   // [2][BM]
    int64_t *colB = rowA + 2 * T::BM;                                    // [2][BN]
    int64_t *colD = colB + 2 * T::BN;                                    // [2][BN]
    int64_t *koffA = colD + 2 * T::BN;
    int64_t *koffB = koffA + kKoffCap;
    uint64_t *bars = reinterpret_cast<uint64_t *>(koffB + kKoffCap);
    unsigned *tmem_slot = reinterpret_cast<unsigned *>(bars + T::NUM_BARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const unsigned raw0 = static_cast<unsigned>(__cvta_generic_to_shared(smem_raw));
    const unsigned tail0 = raw0 + unsigned(T::RAW_STAGES) * T::STAGE_BYTES;
    const unsigned raw_full0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned raw_empty0 = raw_full0 + 8u * T::RAW_STAGES;
    const unsigned tail_full0 = raw_empty0 + 8u * T::RAW_STAGES;
    const unsigned tail_empty0 = tail_full0 + 8u * T::TAIL_STAGES;
    const unsigned accum_full0 = tail_empty0 + 8u * T::TAIL_STAGES;      // [2]
    const unsigned accum_empty0 = accum_full0 + 16u;                     // [2]
    const unsigned producer_sync0 = accum_empty0 + 16u;                  // [2]
    const unsigned epilogue_sync0 = producer_sync0 + 16u;                // [2]

    const int tid = threadIdx.x, warp = tid >> 5;
    const int64_t total = int64_t(p.tiles_m) * p.tiles_n * p.Bt;         // split_k == 1 on this path
    const int num_kt = int((p.K + T::BK - 1) / T::BK);                   // sub-stages of a tile
    const int num_st = (num_kt + T::SUBS - 1) / T::SUBS;                 // stages of a tile
    const bool staged = p.K <= kKoffCap;
    const bool coords_staged = 5 * num_kt <= 2 * kKoffCap;

    // ---- set-up: k offsets, barriers, tensor memory ----
    {
        if (staged)
            for (int i = tid; i < int(p.K); i += T::THREADS) {
                if (!T::A_TMA) koffA[i] = p.offA_k[i];
                koffB[i] = p.offB_k[i];
            }
        // bulk-copy variants: the stages' box coordinates take the place of the M side's k offsets
        if (T::A_TMA && coords_staged)
            for (int i = tid; i < 5 * num_kt; i += T::THREADS) reinterpret_cast<int32_t *>(koffA)[i] = p.tmaA_coord_k[i];
        if (tid == 0) {
            for (int s = 0; s < T::RAW_STAGES; ++s) {
                mbar_init(raw_full0 + 8u * s, T::PRODUCER_THREADS + (T::A_TMA ? 1 : 0));   // + the bulk copy's issuer
                mbar_init(raw_empty0 + 8u * s, 1);
            }
            for (int s = 0; s < T::TAIL_STAGES; ++s) {
                mbar_init(tail_full0 + 8u * s, T::CONVERTER_THREADS);
                mbar_init(tail_empty0 + 8u * s, 1);
            }
            for (int b = 0; b < 2; ++b) {
                mbar_init(accum_full0 + 8u * b, 1);
                mbar_init(accum_empty0 + 8u * b, T::EPILOGUE_THREADS);
                mbar_init(producer_sync0 + 8u * b, T::PRODUCER_THREADS);
                mbar_init(epilogue_sync0 + 8u * b, T::EPILOGUE_THREADS);
            }
            mbar_init(epilogue_sync0 + 16u, 1);      // drain

            *abort_flag = 0;
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        if (warp == T::MMA_WARP) {               // the MMA warp owns the tensor-memory allocation
            tmem_alloc(static_cast<unsigned>(__cvta_generic_to_shared(tmem_slot)), T::TMEM_COLS);
            tmem_relinquish();
        }
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = *tmem_slot;

    if (warp < T::EPILOGUE_WARPS) {
        // ------------------------------------------------------------- epilogue
        // warp w reads tensor-memory lanes 32 w .. 32 w + 31: thread tid owns row tid of the tile
        float *D = static_cast<float *>(p.D);
        const float *C = static_cast<const float *>(p.C);
        const float alpha = float(p.alpha[0]), beta = float(p.beta[0]);
        int n = 0;
#pragma unroll 1
        for (int64_t work = blockIdx.x; work < total; work += gridDim.x, ++n) {
            const TileCoords tc = tile_coords_at<T::BM, T::BN, T::BK>(p, work);
            const int buf = n & 1;
            const unsigned parity = unsigned(n >> 1) & 1u;
            int64_t *cD = colD + buf * T::BN;
            for (int i = tid; i < T::BN; i += T::EPILOGUE_THREADS) cD[i] = i < tc.cols_valid ? p.offD_n[tc.n0 + i] : 0;
            const bool row_ok = tid < tc.rows_valid;
            const int64_t ro = row_ok ? p.offD_m[tc.m0 + tid] + p.offD_h[tc.h] : 0;
            if (!umma_group_sync(epilogue_sync0 + 8u * buf, parity, abort_flag, p.error_word, p.poll_limit)) break;
            if (!mbar_wait_bounded(accum_full0 + 8u * buf, parity, abort_flag, p.error_word, kErrAccumWait, p.poll_limit)) break;
            tc_fence_after();
            const unsigned tacc = tmem_base + (unsigned(warp * 32) << 16) + unsigned(buf * T::ACC_COLS);
#pragma unroll 1
            for (int c0 = 0; c0 < T::BN; c0 += 16) {
                unsigned r[16];
                tmem_load16(tacc + unsigned(c0), r);
                tmem_load_wait();
                float cv[16];
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    cv[j] = (p.use_c && row_ok && c0 + j < tc.cols_valid && BTC_IN_SPAN(p.spans, 2, ro + cD[c0 + j], 1)) ? C[ro + cD[c0 + j]] : 0.f;
#pragma unroll
                for (int j = 0; j < 16; ++j)
                    if (row_ok && c0 + j < tc.cols_valid && BTC_IN_SPAN(p.spans, 2, ro + cD[c0 + j], 1)) {
                        float v = alpha * __uint_as_float(r[j]);
                        if (p.use_c) v += beta * cv[j];
                        D[ro + cD[c0 + j]] = v;
                    }
            }
            tc_fence_before();
            mbar_arrive(accum_empty0 + 8u * buf);    // this accumulator may be overwritten
        }
    } else if (warp < T::EPILOGUE_WARPS + T::CONVERTER_WARPS) {
        // ------------------------------------------------------------- converters
        const int ct = (tid - T::EPILOGUE_THREADS) % T::CONVERTER_THREADS;
        const int group = (tid - T::EPILOGUE_THREADS) / T::CONVERTER_THREADS;
        bool ok = true;
        int g = 0;                                   // stage counter across tiles
#pragma unroll 1
        for (int64_t work = blockIdx.x; ok && work < total; work += gridDim.x) {
#pragma unroll 1
            for (int st = 0; st < num_st; ++st, ++g) {
                if (T::CONVERTER_GROUPS > 1 && g % T::CONVERTER_GROUPS != group) continue;   // another group's stage
                const int s = g % T::RAW_STAGES, t = g % T::TAIL_STAGES;
                if (!mbar_wait_bounded(raw_full0 + 8u * s, unsigned(g / T::RAW_STAGES) & 1u, abort_flag, p.error_word, kErrFullWait, p.poll_limit)) {
                    ok = false;
                    break;
                }
                if (g >= T::TAIL_STAGES &&
                    !mbar_wait_bounded(tail_empty0 + 8u * t, unsigned(g / T::TAIL_STAGES - 1) & 1u, abort_flag, p.error_word, kErrTailEmptyWait, p.poll_limit)) {
                    ok = false;
                    break;
                }
#pragma unroll
                for (int sub = 0; sub < T::SUBS; ++sub) {
                if (st * T::SUBS + sub >= num_kt) break;     // a tile's last stage may hold fewer sub-stages
                const unsigned raw_stage = raw0 + unsigned(s) * T::STAGE_BYTES + unsigned(sub) * T::SUB_BYTES;
                if (T::A_TMEM) {
                    // M-side operand: this thread owns row ct of the tile = lane ct of tensor memory.
                    // It reads the row's 32 k from the raw tile (both layouts give conflict-free
                    // reads with consecutive lanes on consecutive rows), and writes the raw values
                    // (head: the tensor core ignores the low 13 bits) and the tails to the stage's
                    // 32 + 32 tensor-memory columns.
                    // A bulk-copied box is plain: rows of BK k (k contiguous; 128-byte rows carry
                    // the copy's 128-byte swizzle, which is the layout of piece_kmajor; 96-byte rows
                    // are unswizzled and lanes 4-7 of each quarter-warp start one 16-byte chunk
                    // later so that the quarter's eight reads hit distinct banks), or BK columns of
                    // 128 rows (rows contiguous).
                    float x[T::BK], lo[T::BK];
                    if (p.dirA == 1) {
                        if (T::A_TMA && T::BK != 32) {
                            constexpr int CH = T::BK / 4;
                            const int rot = (ct >> 2) & 1;
                            float y[T::BK];
#pragma unroll
                            for (int c = 0; c < CH; ++c) {
                                const int cc = c + rot < CH ? c + rot : c + rot - CH;
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                             : "=f"(y[4 * c]), "=f"(y[4 * c + 1]), "=f"(y[4 * c + 2]), "=f"(y[4 * c + 3])
                                             : "r"(raw_stage + unsigned(ct * (T::BK * 4) + cc * 16)) : "memory");
                            }
#pragma unroll
                            for (int c = 0; c < CH; ++c)       // chunk c was read into slot c - rot
#pragma unroll
                                for (int e = 0; e < 4; ++e) x[4 * c + e] = rot ? y[4 * ((c + CH - 1) % CH) + e] : y[4 * c + e];
                        } else {
#pragma unroll
                            for (int c = 0; c < T::BK / 4; ++c)
                                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                             : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                                             : "r"(raw_stage + piece_kmajor<T::BM>(ct, 4 * c)) : "memory");
                        }
                    } else {
#pragma unroll
                        for (int k = 0; k < T::BK; ++k)
                            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x[k])
                                         : "r"(raw_stage + (T::A_TMA ? unsigned((k * T::BM + ct) * 4) : piece_mnmajor<T::BM>(ct, k))) : "memory");
                    }
#pragma unroll
                    for (int k = 0; k < T::BK; ++k) lo[k] = x[k] - __uint_as_float(__float_as_uint(x[k]) & 0xffffe000u);
                    const unsigned ta = tmem_base + (unsigned(ct & ~31) << 16) + unsigned(2 * T::ACC_COLS + t * T::A_COLS + sub * T::A_SUB_COLS);
                    if constexpr (T::BK == 32) {
                        tmem_store32(ta, x);
                        tmem_store32(ta + 32u, lo);
                    } else {
#pragma unroll
                        for (int j = 0; j < T::KSTEPS; ++j) {
                            tmem_store8(ta + 8u * j, x + 8 * j);
                            tmem_store8(ta + unsigned(T::BK) + 8u * j, lo + 8 * j);
                        }
                    }
                }
                const unsigned src = raw_stage + (T::A_TMEM ? T::A_BYTES : 0) + unsigned(ct) * 16u;
                const unsigned dst = tail0 + unsigned(t) * T::TAIL_BYTES + unsigned(sub) * T::TAIL_SUB_BYTES + unsigned(ct) * 16u;
                constexpr unsigned STEP = 16u * T::CONVERTER_THREADS;
                constexpr int CHUNK = T::PIECES % 8 == 0 ? 8 : T::PIECES % 7 == 0 ? 7 : T::PIECES % 6 == 0 ? 6 : 4;   // loads in flight per thread
                static_assert(T::PIECES % CHUNK == 0, "pieces must divide into chunks");
                // with fewer than 32 k per stage a rows-contiguous N-side tile fills only the front
                // of its place (whole k atoms); a k-contiguous one is spread over all its 128-byte rows
                const int pieces_used = (T::BK == 32 || p.dirB == 1) ? T::PIECES * T::CONVERTER_THREADS : T::BN * T::BK / 4;
#pragma unroll
                for (int i0 = 0; i0 < T::PIECES; i0 += CHUNK) {
                    float x[CHUNK][4];
#pragma unroll
                    for (int i = 0; i < CHUNK; ++i)
                        if (T::BK == 32 || (i0 + i) * T::CONVERTER_THREADS + ct < pieces_used)
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(x[i][0]), "=f"(x[i][1]), "=f"(x[i][2]), "=f"(x[i][3]) : "r"(src + unsigned(i0 + i) * STEP) : "memory");
#pragma unroll
                    for (int i = 0; i < CHUNK; ++i) {
                        if (T::BK != 32 && (i0 + i) * T::CONVERTER_THREADS + ct >= pieces_used) continue;
                        float lo[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e) lo[e] = x[i][e] - __uint_as_float(__float_as_uint(x[i][e]) & 0xffffe000u);
                        asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + unsigned(i0 + i) * STEP), "f"(lo[0]), "f"(lo[1]), "f"(lo[2]), "f"(lo[3]) : "memory");
                    }
                }
                }   // sub-stages
                if (T::A_TMEM) {
                    tmem_store_wait();           // the operand columns are written ...
                    tc_fence_before();           // ... and ordered before the arrival below
                }
                proxy_fence_async();             // the tensor core reads both stages through the async proxy
                mbar_arrive(tail_full0 + 8u * t);
            }
        }
    } else if (warp < T::MMA_WARP) {
        // ------------------------------------------------------------- producers
        const int pt = tid - T::EPILOGUE_THREADS - 32 * T::CONVERTER_WARPS;
        bool ok = true;
        int g = 0, n = 0;
#pragma unroll 1
        for (int64_t work = blockIdx.x; ok && work < total; work += gridDim.x, ++n) {
            const TileCoords tc = tile_coords_at<T::BM, T::BN, T::BK>(p, work);
            const int buf = n & 1;
            int64_t *rA = rowA + buf * T::BM, *cB = colB + buf * T::BN;
            {
                const int64_t hA = p.offA_h[tc.h], hB = p.offB_h[tc.h];
                if (!T::A_TMA)
                    for (int i = pt; i < T::BM; i += T::PRODUCER_THREADS) rA[i] = i < tc.rows_valid ? p.offA_m[tc.m0 + i] + hA : 0;
                for (int i = pt; i < T::BN; i += T::PRODUCER_THREADS) cB[i] = i < tc.cols_valid ? p.offB_n[tc.n0 + i] + hB : 0;
            }
            if (!umma_group_sync(producer_sync0 + 8u * buf, unsigned(n >> 1) & 1u, abort_flag, p.error_word, p.poll_limit)) break;
            const UmmaOperand opA = {static_cast<const float *>(p.A), rA, staged ? koffA : p.offA_k, tc.rows_valid, 0, p.K, p.dirA, p.vecA, &p.spans, 0};
            const UmmaOperand opB = {static_cast<const float *>(p.B), cB, staged ? koffB : p.offB_k, tc.cols_valid, 0, p.K, p.dirB, p.vecB, &p.spans, 1};
            UmmaProducerLane<T::BM> la;
            UmmaProducerLane<T::BN> lb;
            if (!T::A_TMA) umma_producer_init<T::BM>(la, opA, pt);
            umma_producer_init<T::BN>(lb, opB, pt);
            int box0[5] = {0, 0, 0, 0, 0};           // bulk copy: the box origin of this tile at stage 0
            if (T::A_TMA && pt == 0) {
                const int32_t *cm = p.tmaA_coord_m + (tc.m0 / T::BM) * 5, *ch = p.tmaA_coord_h + tc.h * 5;
#pragma unroll
                for (int d = 0; d < 5; ++d) box0[d] = cm[d] + ch[d];
            }
            // offsets of the first stage; inside the loop those of the next stage are looked up
            // before this stage's copies are issued
            UmmaStageOffsets sa = {0, 0, false, false}, sb = sa, sa_next = sa, sb_next = sa;
            if (!T::A_TMA && opA.vec == 4) sa_next = umma_lookup<T::BM>(la, opA, 0);
            if (opB.vec == 4) sb_next = umma_lookup<T::BN, T::BK>(lb, opB, 0);
#pragma unroll 1
            for (int st_i = 0; st_i < num_st; ++st_i, ++g) {
                const int s = g % T::RAW_STAGES;
                if (T::SUBS == 1) {
                    sa = sa_next; sb = sb_next;
                    if (st_i + 1 < num_st) {
                        if (!T::A_TMA && opA.vec == 4) sa_next = umma_lookup<T::BM>(la, opA, int64_t(st_i + 1) * T::BK);
                        if (opB.vec == 4) sb_next = umma_lookup<T::BN, T::BK>(lb, opB, int64_t(st_i + 1) * T::BK);
                    }
                }
                if (g >= T::RAW_STAGES &&
                    !mbar_wait_bounded(raw_empty0 + 8u * s, unsigned(g / T::RAW_STAGES - 1) & 1u, abort_flag, p.error_word, kErrEmptyWait, p.poll_limit)) {
                    ok = false;
                    break;
                }
                const int subs_here = num_kt - st_i * T::SUBS < T::SUBS ? num_kt - st_i * T::SUBS : T::SUBS;
                if (T::A_TMA && pt == 0) mbar_arrive_expect_tx(raw_full0 + 8u * s, unsigned(T::A_BYTES) * unsigned(subs_here));
#pragma unroll
                for (int sub = 0; sub < T::SUBS; ++sub) {
                    if (sub >= subs_here) break;
                    const int kt = st_i * T::SUBS + sub;
                    const unsigned st = raw0 + unsigned(s) * T::STAGE_BYTES + unsigned(sub) * T::SUB_BYTES;
                    const int64_t k0 = int64_t(kt) * T::BK;
                    if (T::SUBS > 1) {
                        if (!T::A_TMA && opA.vec == 4) sa = umma_lookup<T::BM>(la, opA, k0);
                        if (opB.vec == 4) sb = umma_lookup<T::BN, T::BK>(lb, opB, k0);
                    }
                    if (T::A_TMA) {
                        if (pt == 0) {
                            const int32_t *ck = (coords_staged ? reinterpret_cast<const int32_t *>(koffA) : p.tmaA_coord_k) + kt * 5;
                            tma_load_box(st, &tmapA, raw_full0 + 8u * s, box0[0] + ck[0], box0[1] + ck[1], box0[2] + ck[2],
                                         box0[3] + ck[3], box0[4] + ck[4]);
                        }
                    } else {
                        umma_produce<T::BM>(st, la, opA, k0, sa);
                    }
                    umma_produce<T::BN, T::BK>(st + T::A_BYTES, lb, opB, k0, sb);
                }
                mbar_arrive_on_copies(raw_full0 + 8u * s);
            }
        }
        cp_async_wait_all();
    } else {
        // ------------------------------------------------------------- MMA warp
        constexpr unsigned IDESC_KK = umma_instr_desc(T::BN, false, false);
        constexpr unsigned IDESC_MK = umma_instr_desc(T::BN, true, false);
        constexpr unsigned IDESC_KM = umma_instr_desc(T::BN, false, true);
        constexpr unsigned IDESC_MM = umma_instr_desc(T::BN, true, true);
        const bool a_mn = !T::A_TMEM && p.dirA == 0, b_mn = p.dirB == 0;   // an operand in tensor memory is K-major
        const unsigned idesc = a_mn ? (b_mn ? IDESC_MM : IDESC_MK) : (b_mn ? IDESC_KM : IDESC_KK);
        // per operand: layout type, leading / stride byte offsets, start advance of one k-step (8 k)
        const unsigned a_lay = a_mn ? 1u : 2u, a_lbo = a_mn ? 512u : 16u, a_sbo = a_mn ? 16u * T::BM : 1024u;
        const unsigned b_lay = b_mn ? 1u : 2u, b_lbo = b_mn ? 512u : 16u, b_sbo = b_mn ? 16u * T::BN : 1024u;
        const unsigned a_step = a_mn ? 32u * T::BM : 32u, b_step = b_mn ? 32u * T::BN : 32u;   // two k-atoms, or 8 k of a row
        const bool leader = elect_one();
        bool ok = true;
        int g = 0, n = 0;
#pragma unroll 1
        for (int64_t work = blockIdx.x; ok && work < total; work += gridDim.x, ++n) {
            const int buf = n & 1;
            if (n >= 2 &&
                !mbar_wait_bounded(accum_empty0 + 8u * buf, unsigned((n >> 1) - 1) & 1u, abort_flag, p.error_word, kErrAccumWait, p.poll_limit))
                break;
            tc_fence_after();
            const unsigned tacc = tmem_base + unsigned(buf * T::ACC_COLS);
#pragma unroll 1
            for (int st = 0; st < num_st; ++st, ++g) {
                const int s = g % T::RAW_STAGES, t = g % T::TAIL_STAGES;
                if (!mbar_wait_bounded(tail_full0 + 8u * t, unsigned(g / T::TAIL_STAGES) & 1u, abort_flag, p.error_word, kErrTailFullWait, p.poll_limit)) {
                    ok = false;
                    break;
                }
                tc_fence_after();
                if (leader) {
#pragma unroll
                    for (int sub = 0; sub < T::SUBS; ++sub) {
                    if (st * T::SUBS + sub >= num_kt) break;
                    const unsigned a_hi = raw0 + unsigned(s) * T::STAGE_BYTES + unsigned(sub) * T::SUB_BYTES, b_hi = a_hi + T::A_BYTES;
                    const unsigned a_lo = tail0 + unsigned(t) * T::TAIL_BYTES + unsigned(sub) * T::TAIL_SUB_BYTES, b_lo = a_lo + T::TAIL_B_OFFSET;
                    const unsigned ta = tmem_base + unsigned(2 * T::ACC_COLS + t * T::A_COLS + sub * T::A_SUB_COLS);   // head columns, tail BK further
#pragma unroll
                    for (int j = 0; j < T::KSTEPS; ++j) {
                        const uint64_t dbh = umma_smem_desc(b_hi + j * b_step, b_lbo, b_sbo, b_lay);
                        const uint64_t dbl = umma_smem_desc(b_lo + j * b_step, b_lbo, b_sbo, b_lay);
                        const unsigned acc_in = (st > 0 || sub > 0 || j > 0) ? 1u : 0u;
                        if (T::A_TMEM) {
                            umma_tf32_ts(tacc, ta + unsigned(T::BK) + 8u * j, dbh, idesc, acc_in);
                            umma_tf32_ts(tacc, ta + 8u * j, dbl, idesc, 1u);
                            umma_tf32_ts(tacc, ta + 8u * j, dbh, idesc, 1u);
                        } else {
                            const uint64_t dah = umma_smem_desc(a_hi + j * a_step, a_lbo, a_sbo, a_lay);
                            const uint64_t dal = umma_smem_desc(a_lo + j * a_step, a_lbo, a_sbo, a_lay);
                            umma_tf32(tacc, dal, dbh, idesc, acc_in);
                            umma_tf32(tacc, dah, dbl, idesc, 1u);
                            umma_tf32(tacc, dah, dbh, idesc, 1u);
                        }
                    }
                    }   // sub-stages
                    umma_commit(raw_empty0 + 8u * s);    // fire when these MMAs have read the stages
                    umma_commit(tail_empty0 + 8u * t);
                    if (st + 1 == num_st) umma_commit(accum_full0 + 8u * buf);
                }
                __syncwarp();
            }
        }
        tc_fence_before();
    }

    // ---- common tail: every role arrives here, also after an abort ----
    // After an abort work may still be in flight that must not outlive the CTA: asynchronous copies
    // (the producers have waited for theirs above), tensor-core instructions (drained below through a
    // commit on a barrier of its own, with a bounded wait) and, in the bulk-copy variants, box copies
    // whose completion barrier may never fire because some producers have left: those land within a
    // few microseconds, so the CTA lingers that long before it gives up its shared memory.
    if (T::A_TMA && *abort_flag && tid == T::EPILOGUE_THREADS + 32 * T::CONVERTER_WARPS) __nanosleep(20000);
    __syncthreads();
    if (warp == T::MMA_WARP) {
        if (*abort_flag) {
            const unsigned drain = epilogue_sync0 + 16u;
            if (elect_one()) umma_commit(drain);
            __syncwarp();
            for (unsigned n = 0; n < (1u << 16) && !mbar_try_wait(drain, 0u); ++n) { }
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

}  // namespace btc

// Bandwidth-bound fp32 contraction for short contracted extents (K <= 64) on the 5th-generation
// tensor cores: the low-intensity path of the contraction D = alpha op(A) op(B) + beta op(C)
// (Eq. (case2)) for shapes such as tensor-network contractions of many small modes, where the
// result is far larger than the inputs and the kernel's job is to stream D at memory speed.
//
// All of K fits one shared-memory tile, so there is no k loop and no stage ring along k.
// Persistent CTAs (one per SM) each take a contiguous range of the 128 x 128 output tiles, ordered
// (batch entry, tile row, tile column) with the column fastest, so that consecutive tiles of a CTA
// share their M-side operand tile ("strip"), which is fetched and converted once per strip.
//   loaders     fetch the operand tiles with 16-byte asynchronous copies enumerated IN MEMORY
//               ORDER: the host sorts the tile's 16-byte pieces by address once per operation
//               ("piece order" tables), so a warp's 32 copies cover whole 128-byte lines even when
//               free and contracted modes interleave in memory with runs of only 16 bytes.
//   converters  3xTF32 split (x = x_hi + x_lo; a b ~ a_lo b_hi + a_hi b_lo + a_hi b_hi, dropped term
//               <= 2^-22 |a||b|).  The M-side tile goes to tensor memory (head and tail, one row per
//               lane); the N-side tile stays in shared memory in the layout the tensor core reads
//               (its raw form is the head: the tensor core ignores the low 13 mantissa bits) and its
//               tail is written to a second buffer.
//   MMA warp    one elected lane issues ceil(K / 8) x 3 tcgen05.mma (M 128, N 128, K 8) per tile into
//               one of two accumulators in tensor memory.
//   epilogue    four warps (one tensor-memory lane quarter each, one row of the tile per lane) read the
//               accumulator and write D straight from registers, applying alpha / beta / C on the way:
//               16-byte stores of four consecutive columns when those are contiguous in D (the host
//               then puts D's smallest-stride label on the column side), element stores of 32
//               consecutive rows per warp otherwise.
// Every wait is bounded (poll limit, then error word + CTA abort flag, no trap); all roles meet
// at the common tail, where the allocating warp frees the tensor memory.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"
#include "tile_common.cuh"
#include "tiled_umma_tf32x3_kernel.cuh"
#include "skinny_layout.h"

namespace btc {

struct SkinnyTile {
    static constexpr int BM = 128, BN = 128, KMAX = 64;
    // the N-side tiles wait in a ring of raw stages (filled up to three tiles ahead of the tensor core, to ride out
    // the memory latency); their tails are made just in time into a shorter ring
    static constexpr int RAW_STAGES = 3, LO_STAGES = 2;
    static constexpr int EPILOGUE_WARPS = 4, CONVERTER_WARPS = 4, LOADER_WARPS = 4;
    static constexpr int GROUP_THREADS = 128;
    static constexpr int MMA_WARP = EPILOGUE_WARPS + CONVERTER_WARPS + LOADER_WARPS;
    static constexpr int THREADS = 32 * (MMA_WARP + 1);
    static constexpr int A_BYTES = BM * KMAX * 4;            // raw M-side tile (layout of our own: never read by the tensor core)
    static constexpr int B_BYTES = BN * KMAX * 4;            // N-side tile: two blocks of 32 k in the tensor core's layout
    static constexpr int B_BLOCK_BYTES = BN * 128;           // one block of 32 k
    static constexpr int PIECES = BM * KMAX / 4;             // 16-byte pieces of a full operand tile
    static constexpr int PER_THREAD = PIECES / GROUP_THREADS;
    static constexpr int ACC_COLS = 128, A_COLS = 2 * KMAX;  // tensor-memory columns: accumulator; head + tail of the M side
    static constexpr int TMEM_COLS = 512;                    // 2 accumulators + 2 M-side operand buffers
    static constexpr int NUM_BARS = 24;
    static constexpr int SPLIT_COL = 64;                     // columns below: epilogue warps; from here on: the converter warps, between conversions
    // N-side raw[3] | N-side tail[2] | M-side raw | row / column offsets | k offsets | piece tables | barriers | slot, abort
    static constexpr size_t SMEM_BYTES = size_t(RAW_STAGES + LO_STAGES) * B_BYTES + A_BYTES +
                                         size_t(2 * BM + RAW_STAGES * BN + 2 * KMAX) * 8 + size_t(2 * PIECES) * 4 +
                                         size_t(NUM_BARS) * 8 + 16 + 1024;
};

// debug builds (-DBTC_STAMPS -DBTC_EVENTS): CTA 0 records the SM clock at eight events of its first 64 tiles
#if defined(BTC_STAMPS) && defined(BTC_EVENTS)
#define BTC_EVENT(p, who, ev, i) do { if ((who) && (p).stamps && blockIdx.x == 0 && (i) < 64) (p).stamps[2048 + (ev) * 64 + (i)] = clock64(); } while (0)
#else
#define BTC_EVENT(p, who, ev, i) do { } while (0)
#endif
#if defined(BTC_STAMPS) && defined(BTC_EVENTS_EPI)
#define BTC_EPI_EVENT(p, who, ev, i) do { if ((who) && (p).stamps && blockIdx.x == 0 && (i) < 64) (p).stamps[2048 + (ev) * 64 + (i)] = clock64(); } while (0)
#else
#define BTC_EPI_EVENT(p, who, ev, i) do { } while (0)
#endif

constexpr int kErrSkinnyLoad = 8, kErrSkinnyConvert = 9, kErrSkinnyMma = 10, kErrSkinnyEpilogue = 11;

// One operand tile: every loader thread copies its pieces (entries pt, pt + 128, ... of the piece
// order), eight look-ups first, then their eight copies.  `table` (shared memory) holds per piece, in
// piece order: bits 0-10 the piece (see skinny_a_pos / skinny_b_pos), bit 11 its k < K, bits 12-31 (signed)
// its offset relative to the tile's first row in units of four elements (regular operands only).
template <bool IS_A>
__device__ __forceinline__ void skinny_load_tile(unsigned tile, const float *g, const int64_t *row_off, const int64_t *koff,
                                                 const unsigned *table, int pieces, int dir, int rows_valid, int pt,
                                                 const OffsetSpans &spans, int which)
{
#pragma unroll 1
    for (int e0 = pt; e0 < pieces; e0 += 8 * SkinnyTile::GROUP_THREADS) {
        int64_t off[8];
        unsigned dst[8];
        bool valid[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = e0 + j * SkinnyTile::GROUP_THREADS;
            const unsigned pk = e < pieces ? table[e] : 0u;
            int row, k;
            dst[j] = IS_A ? skinny_a_pos(dir, pk & 2047u, row, k) : skinny_b_pos(dir, pk & 2047u, row, k);
            valid[j] = ((pk >> 11) & 1u) && row < rows_valid;
            off[j] = valid[j] ? row_off[row] + koff[k] : 0;
            if (valid[j] && !BTC_IN_SPAN(spans, which, off[j], 4)) { valid[j] = false; off[j] = 0; }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (e0 + j * SkinnyTile::GROUP_THREADS < pieces) cp_async_bytes<16>(tile + dst[j], g + off[j], valid[j]);
    }
}
// The same for a regular operand (every tile's rows lie relative to its first row as tile 0's do):
// `base` is the offset of the tile's first row, the table gives the rest; no offset arrays are needed.
template <bool IS_A>
__device__ __forceinline__ void skinny_load_tile_regular(unsigned tile, const float *g, int64_t base, const unsigned *table, int pieces,
                                                         int dir, int rows_valid, int pt, const OffsetSpans &spans, int which)
{
#pragma unroll 1
    for (int e0 = pt; e0 < pieces; e0 += 8 * SkinnyTile::GROUP_THREADS) {
        unsigned q[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            const int e = e0 + j * SkinnyTile::GROUP_THREADS;
            q[j] = e < pieces ? table[e] : 0u;
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            int row, k;
            const unsigned dst = IS_A ? skinny_a_pos(dir, q[j] & 2047u, row, k) : skinny_b_pos(dir, q[j] & 2047u, row, k);
            const int64_t off = base + 4 * int64_t(int(q[j]) >> 12);
            bool valid = ((q[j] >> 11) & 1u) && row < rows_valid;
            valid = valid && BTC_IN_SPAN(spans, which, off, 4);
            if (e0 + j * SkinnyTile::GROUP_THREADS < pieces) cp_async_bytes<16>(tile + dst, g + (valid ? off : 0), valid);
        }
    }
}

struct SkinnyWork {
    int64_t h;
    int mt, nt;
    int64_t m0, n0;
    int rows_valid, cols_valid;
};
__device__ __forceinline__ void skinny_work_fill(const TiledParams &p, SkinnyWork &w)
{
    w.m0 = int64_t(w.mt) * SkinnyTile::BM;
    w.n0 = int64_t(w.nt) * SkinnyTile::BN;
    w.rows_valid = int(imin64(SkinnyTile::BM, p.M - w.m0));
    w.cols_valid = int(imin64(SkinnyTile::BN, p.N - w.n0));
}
// tile t of the list (batch entry, tile row, tile column), column fastest
__device__ __forceinline__ SkinnyWork skinny_work_at(const TiledParams &p, int64_t t)
{
    SkinnyWork w;
    w.nt = int(t % p.tiles_n);
    const int64_t q = t / p.tiles_n;
    w.mt = int(q % p.tiles_m);
    w.h = q / p.tiles_m;
    skinny_work_fill(p, w);
    return w;
}
// the tile after w (no divisions: every role steps through its tiles with this)
__device__ __forceinline__ SkinnyWork skinny_work_next(const TiledParams &p, const SkinnyWork &w)
{
    SkinnyWork n = w;
    if (++n.nt == p.tiles_n) {
        n.nt = 0;
        if (++n.mt == p.tiles_m) {
            n.mt = 0;
            ++n.h;
        }
    }
    skinny_work_fill(p, n);
    return n;
}

// What one thread keeps to write its row of the accumulators to D.  Thread `row` owns row `row` of every
// tile (tensor-memory lane `row`).  Two ways to write:
//   vecn (groups of four consecutive columns are 16 contiguous, aligned bytes of D): one 16-byte store
//        per group straight from the accumulator registers.  The host puts D's smallest-stride label on
//        the column side when its contiguous runs are short, so that the few lanes whose rows are
//        neighbours in D complete whole 128-byte lines between them.
//   otherwise: one element per store; a warp's store of one column = 32 consecutive rows.
// Offsets: row part from the tables (fetched when a strip starts), column part either from the constant
// bank (regular columns: offset of the tile's first column + skinny_col_rel) or from per-lane table
// entries handed round by shuffle (vecn: lane l holds column group l; else co[c] = column 32 c + lane).
// Both are fetched one tile ahead of their use.
struct SkinnyStore {
    float *D;
    const float *C;
    float alpha, beta;
    bool vecn, dreg;
    int row, lane;
    int64_t ro, ro_next, co_next[4];
    bool row_ok, row_ok_next;

    __device__ __forceinline__ void init(const TiledParams &p, int row_, int lane_)
    {
        D = static_cast<float *>(p.D);
        C = static_cast<const float *>(p.C);
        alpha = float(p.alpha[0]); beta = float(p.beta[0]);
        vecn = p.skinny_vec_n == 4; dreg = p.skinny_d_regular != 0;
        row = row_; lane = lane_;
        ro = ro_next = 0; row_ok = row_ok_next = false;
        co_next[0] = co_next[1] = co_next[2] = co_next[3] = 0;
    }
    // start fetching what tile wk needs; `strip_start`: wk is the first tile of a strip for this CTA
    __device__ __forceinline__ void fetch(const TiledParams &p, const SkinnyWork &wk, bool strip_start)
    {
        if (strip_start) {
            row_ok_next = row < wk.rows_valid;
            ro_next = row_ok_next ? p.offD_m[wk.m0 + row] + p.offD_h[wk.h] : 0;
        }
        if (dreg) {
            co_next[0] = p.offD_n[wk.n0];
        } else if (vecn) {
            co_next[0] = 4 * lane < wk.cols_valid ? p.offD_n[wk.n0 + 4 * lane] : 0;
        } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) co_next[c] = (c * 32 + lane < wk.cols_valid) ? p.offD_n[wk.n0 + c * 32 + lane] : 0;
        }
    }
    // Columns [c_begin, c_end) (multiples of 32) of the accumulator at `tacc` (this warp's lane quarter)
    // -> D.  `co` = the column offsets fetched for this tile.  Arrives on `done_bar` as soon as the
    // columns are in registers.
    __device__ __forceinline__ void tile(const TiledParams &p, const SkinnyWork &w, unsigned tacc, int c_begin, int c_end,
                                         unsigned done_bar, const int64_t (&co)[4])
    {
#pragma unroll 1
        for (int c0 = c_begin; c0 < c_end; c0 += 32) {       // rolled: keeps the code small
            unsigned r[32];
            tmem_load16(tacc + unsigned(c0), *reinterpret_cast<unsigned (*)[16]>(&r[0]));
            tmem_load16(tacc + unsigned(c0 + 16), *reinterpret_cast<unsigned (*)[16]>(&r[16]));
            tmem_load_wait();
            if (c0 + 32 == c_end) {                  // this thread's share of the accumulator is in registers
                tc_fence_before();
                mbar_arrive(done_bar);
            }
            const int cols_here = w.cols_valid - c0;         // valid columns from c0 on (may be <= 0)
            if (vecn) {
                int64_t off[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    off[q] = ro + (dreg ? co[0] + p.skinny_col_rel[c0 + 4 * q] : __shfl_sync(0xffffffffu, co[0], (c0 >> 2) + q));
                float4 v[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    v[q] = make_float4(alpha * __uint_as_float(r[4 * q]), alpha * __uint_as_float(r[4 * q + 1]),
                                       alpha * __uint_as_float(r[4 * q + 2]), alpha * __uint_as_float(r[4 * q + 3]));
                if (p.use_c) {
#pragma unroll
                    for (int q0 = 0; q0 < 8; q0 += 4) {
                        float4 cv[4];
#pragma unroll
                        for (int q = 0; q < 4; ++q)
                            cv[q] = (row_ok && 4 * (q0 + q) < cols_here && BTC_IN_SPAN(p.spans, 2, off[q0 + q], 4))
                                        ? *reinterpret_cast<const float4 *>(C + off[q0 + q]) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            v[q0 + q].x += beta * cv[q].x; v[q0 + q].y += beta * cv[q].y;
                            v[q0 + q].z += beta * cv[q].z; v[q0 + q].w += beta * cv[q].w;
                        }
                    }
                }
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    if (row_ok && 4 * q < cols_here && BTC_IN_SPAN(p.spans, 2, off[q], 4)) *reinterpret_cast<float4 *>(D + off[q]) = v[q];
            } else {
                const int64_t mine = c0 == 0 ? co[0] : c0 == 32 ? co[1] : c0 == 64 ? co[2] : co[3];
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    const int64_t off = ro + (dreg ? co[0] + p.skinny_col_rel[c0 + j] : __shfl_sync(0xffffffffu, mine, j));
                    if (row_ok && j < cols_here && BTC_IN_SPAN(p.spans, 2, off, 1)) {
                        float v = alpha * __uint_as_float(r[j]);
                        if (p.use_c) v += beta * C[off];
                        D[off] = v;
                    }
                }
            }
        }
    }
};

__global__ void __launch_bounds__(SkinnyTile::THREADS, 1) skinny_umma_kernel(const TiledParams p)
{
    using T = SkinnyTile;
    extern __shared__ __align__(16) unsigned char smem_unaligned[];
    unsigned char *smem_raw = smem_unaligned +
        ((1024u - (static_cast<unsigned>(__cvta_generic_to_shared(smem_unaligned)) & 1023u)) & 1023u);
    unsigned char *cursor = smem_raw + size_t(T::RAW_STAGES + T::LO_STAGES) * T::B_BYTES + T::A_BYTES;
    int64_t *rowA = reinterpret_cast<int64_t *>(cursor);                 // [2][BM]
    int64_t *colB = rowA + 2 * T::BM;                                    // [RAW_STAGES][BN]
    int64_t *koffA = colB + T::RAW_STAGES * T::BN;                       // [KMAX]
    int64_t *koffB = koffA + T::KMAX;                                    // [KMAX]
    unsigned *pieceA = reinterpret_cast<unsigned *>(koffB + T::KMAX);    // [PIECES] piece tables
    unsigned *pieceB = pieceA + T::PIECES;                               // [PIECES]
    uint64_t *bars = reinterpret_cast<uint64_t *>(pieceB + T::PIECES);
    unsigned *tmem_slot = reinterpret_cast<unsigned *>(bars + T::NUM_BARS);
    volatile int *abort_flag = reinterpret_cast<volatile int *>(tmem_slot + 1);
    const unsigned braw0 = static_cast<unsigned>(__cvta_generic_to_shared(smem_raw));
    const unsigned blo0 = braw0 + unsigned(T::RAW_STAGES) * T::B_BYTES;
    const unsigned araw = blo0 + unsigned(T::LO_STAGES) * T::B_BYTES;
    const unsigned bar0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned a_full = bar0, a_empty = bar0 + 8u;
    const unsigned raw_full0 = bar0 + 16u, raw_empty0 = raw_full0 + 24u;                      // [3] each
    const unsigned lo_conv0 = raw_empty0 + 24u, lo_empty0 = lo_conv0 + 16u;                   // [2] each
    const unsigned ta_full0 = lo_empty0 + 16u, ta_empty0 = ta_full0 + 16u;                    // [2] each
    const unsigned acc_full0 = ta_empty0 + 16u, acc_empty0 = acc_full0 + 16u;                 // [2] each
    const unsigned loader_sync = acc_empty0 + 16u, drain = loader_sync + 8u;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = int(p.K);
    const int ksteps = (K + 7) / 8, kp = 8 * ksteps;                     // tensor-core steps of 8 k; k padded with zeros
    const int pieces = 32 * kp;                                         // 16-byte pieces of an operand tile in use
    const int64_t total = int64_t(p.tiles_m) * p.tiles_n * p.Bt;
    const int64_t t0 = total * blockIdx.x / gridDim.x, t1 = total * (blockIdx.x + 1) / gridDim.x;

    // ---- set-up: k offsets, barriers, tensor memory ----
    for (int i = tid; i < T::KMAX; i += T::THREADS) {
        koffA[i] = i < K ? p.offA_k[i] : 0;
        koffB[i] = i < K ? p.offB_k[i] : 0;
    }
    for (int e = tid; e < pieces; e += T::THREADS) {
        int row, k;
        unsigned code = p.skinny_orderA[e];
        skinny_a_pos(p.dirA, code, row, k);
        int64_t rel = (row < p.M && k < K) ? p.offA_m[row] - p.offA_m[0] + p.offA_k[k] : 0;
        pieceA[e] = code | (unsigned(k < K) << 11) | (unsigned(int(rel / 4)) << 12);
        code = p.skinny_orderB[e];
        skinny_b_pos(p.dirB, code, row, k);
        rel = (row < p.N && k < K) ? p.offB_n[row] - p.offB_n[0] + p.offB_k[k] : 0;
        pieceB[e] = code | (unsigned(k < K) << 11) | (unsigned(int(rel / 4)) << 12);
    }
    if (tid == 0) {
        mbar_init(a_full, T::GROUP_THREADS);
        mbar_init(a_empty, T::GROUP_THREADS);
        for (int s = 0; s < 2; ++s) {
            mbar_init(lo_conv0 + 8u * s, T::GROUP_THREADS);
            mbar_init(lo_empty0 + 8u * s, 1);
            mbar_init(ta_full0 + 8u * s, T::GROUP_THREADS);
            mbar_init(ta_empty0 + 8u * s, 1);
            mbar_init(acc_full0 + 8u * s, 1);
            mbar_init(acc_empty0 + 8u * s, 2 * T::GROUP_THREADS);
        }
        for (int s = 0; s < T::RAW_STAGES; ++s) {
            mbar_init(raw_full0 + 8u * s, T::GROUP_THREADS);
            mbar_init(raw_empty0 + 8u * s, 1);
        }
        mbar_init(loader_sync, T::GROUP_THREADS);
        mbar_init(drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == T::MMA_WARP) {
        tmem_alloc(static_cast<unsigned>(__cvta_generic_to_shared(tmem_slot)), T::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const unsigned tmem_base = *tmem_slot;
    const unsigned tmem_a0 = tmem_base + 2u * T::ACC_COLS;

    if (warp < T::EPILOGUE_WARPS) {
        // ------------------------------------------------------------- epilogue (first half of the columns)
        SkinnyStore st;
        st.init(p, tid, lane);
        SkinnyWork w = skinny_work_at(p, t0);
        if (t0 < t1) st.fetch(p, w, true);
        long long t_wait = 0, t_work = 0;
        (void)t_wait; (void)t_work;
        BTC_PHASE_BEGIN();
#pragma unroll 1
        for (int64_t t = t0; t < t1; ++t) {
            const int i = int(t - t0), buf = i & 1;
            const SkinnyWork wn = skinny_work_next(p, w);
            if (t == t0 || w.nt == 0) { st.ro = st.ro_next; st.row_ok = st.row_ok_next; }
            int64_t co[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) co[c] = st.co_next[c];
            if (t + 1 < t1) st.fetch(p, wn, wn.nt == 0);
            BTC_PHASE_END(t_work);
            if (!mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(i >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit)) break;
            BTC_PHASE_END(t_wait);
            BTC_EVENT(p, tid == 0, 6, i);
            tc_fence_after();
            st.tile(p, w, tmem_base + (unsigned(warp * 32) << 16) + unsigned(buf * T::ACC_COLS), 0, T::SPLIT_COL, acc_empty0 + 8u * buf, co);
            BTC_EVENT(p, tid == 0, 7, i);
            w = wn;
        }
        BTC_PHASE_END(t_work);
        BTC_PHASE_STORE(p, tid == 0, 0, t_wait);
        BTC_PHASE_STORE(p, tid == 0, 1, t_work);
    } else if (warp < T::EPILOGUE_WARPS + T::CONVERTER_WARPS) {
        // ------------------------------------------------------------- converters
        const int ct = tid - 32 * T::EPILOGUE_WARPS;             // row of the M-side tile = tensor-memory lane
        int sidx = -1;
        long long t_wait = 0, t_work = 0;
        (void)t_wait; (void)t_work;
        // Between conversions these warps also write the second half of the columns of the tile before
        // (its accumulator is complete by then), which doubles the warps that keep stores in flight.
        SkinnyStore st;
        st.init(p, ct, lane);
        SkinnyWork w = skinny_work_at(p, t0), wprev = w;
        int64_t co_prev[4] = {0, 0, 0, 0};
        BTC_PHASE_BEGIN();
#pragma unroll 1
        for (int64_t t = t0; t < t1; ++t) {
            const int i = int(t - t0), s = i & 1;
            const bool new_strip = t == t0 || w.nt == 0;
            st.fetch(p, w, new_strip);                // for this tile's store, one iteration from now
            if (new_strip) {
                ++sidx;
                const int ab = sidx & 1;
                if (!mbar_wait_bounded(a_full, unsigned(sidx) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit)) break;
                if (sidx >= 2 &&
                    !mbar_wait_bounded(ta_empty0 + 8u * ab, unsigned((sidx >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit))
                    break;
                tc_fence_after();
                const unsigned ta = tmem_a0 + unsigned(ab * T::A_COLS) + (unsigned(ct & ~31) << 16);
#pragma unroll
                for (int half = 0; half < 2; ++half) {
                    if (half * 32 >= kp) break;
                    float x[32];
                    if (p.dirA == 0) {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x[k]) : "r"(araw + unsigned((half * 32 + k) * T::BM + ct) * 4u) : "memory");
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                                         : "r"(araw + unsigned(ct) * 256u + (unsigned(((half * 8 + c) ^ ct) & 15) << 4)) : "memory");
                    }
                    tmem_store32(ta + unsigned(half * 32), x);
#pragma unroll
                    for (int k = 0; k < 32; ++k) x[k] -= __uint_as_float(__float_as_uint(x[k]) & 0xffffe000u);
                    tmem_store32(ta + unsigned(T::KMAX + half * 32), x);
                }
                tmem_store_wait();
                tc_fence_before();
                mbar_arrive(ta_full0 + 8u * ab);
                mbar_arrive(a_empty);                 // the raw M-side buffer may be refilled
            }
            BTC_PHASE_END(t_work);
            const int r = i % T::RAW_STAGES;
            if (!mbar_wait_bounded(raw_full0 + 8u * r, unsigned(i / T::RAW_STAGES) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit)) break;
            // the tail stage is free once the tensor core has finished the tile two before this one
            if (i >= 2 && !mbar_wait_bounded(lo_empty0 + 8u * s, unsigned((i >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit)) break;
            BTC_PHASE_END(t_wait);
            BTC_EVENT(p, ct == 0, 2, i);
            // N side: position-independent pass; the raw stage is the head, the tail goes to the same
            // position of the tail stage
            const unsigned src = braw0 + unsigned(r) * T::B_BYTES + unsigned(ct) * 16u;
            const unsigned dst = blo0 + unsigned(s) * T::B_BYTES + unsigned(ct) * 16u;
            const int per = (kp <= 32 ? T::B_BLOCK_BYTES : T::B_BYTES) / 16 / T::GROUP_THREADS;   // 8 or 16 pieces per thread
#pragma unroll
            for (int i0 = 0; i0 < 16; i0 += 8) {
                if (i0 >= per) break;
                float x[8][4];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                 : "=f"(x[q][0]), "=f"(x[q][1]), "=f"(x[q][2]), "=f"(x[q][3]) : "r"(src + unsigned(i0 + q) * 2048u) : "memory");
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    float lo[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) lo[e] = x[q][e] - __uint_as_float(__float_as_uint(x[q][e]) & 0xffffe000u);
                    asm volatile("st.shared.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst + unsigned(i0 + q) * 2048u), "f"(lo[0]), "f"(lo[1]), "f"(lo[2]), "f"(lo[3]) : "memory");
                }
            }
            proxy_fence_async();                      // the tensor core reads both stages through the async proxy
            mbar_arrive(lo_conv0 + 8u * s);
            BTC_EVENT(p, ct == 0, 3, i);
            if (i > 0) {
                const int ip = i - 1, buf = ip & 1;
                if (!mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(ip >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit)) break;
                tc_fence_after();
                st.tile(p, wprev, tmem_base + (unsigned(ct & ~31) << 16) + unsigned(buf * T::ACC_COLS), T::SPLIT_COL, T::BN,
                        acc_empty0 + 8u * buf, co_prev);
            }
            // what was fetched at the top of this iteration belongs to this tile: keep it for the next iteration
#pragma unroll
            for (int c = 0; c < 4; ++c) co_prev[c] = st.co_next[c];
            if (new_strip) { st.ro = st.ro_next; st.row_ok = st.row_ok_next; }
            wprev = w;
            w = skinny_work_next(p, w);
        }
        if (t1 > t0 && !*abort_flag) {                // the last tile's second half
            const int ip = int(t1 - t0) - 1, buf = ip & 1;
            if (mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(ip >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit)) {
                tc_fence_after();
                st.tile(p, wprev, tmem_base + (unsigned(ct & ~31) << 16) + unsigned(buf * T::ACC_COLS), T::SPLIT_COL, T::BN,
                        acc_empty0 + 8u * buf, co_prev);
            }
        }
        BTC_PHASE_END(t_work);
        BTC_PHASE_STORE(p, ct == 0, 2, t_wait);
        BTC_PHASE_STORE(p, ct == 0, 3, t_work);
    } else if (warp < T::MMA_WARP) {
        // ------------------------------------------------------------- loaders
        const int pt = tid - 32 * (T::EPILOGUE_WARPS + T::CONVERTER_WARPS);
        const float *A = static_cast<const float *>(p.A), *B = static_cast<const float *>(p.B);
        int sidx = -1;
        long long t_wait = 0, t_work = 0;
        (void)t_wait; (void)t_work;
        // Regular operands: a tile is addressed by its first row's offset alone, fetched one tile ahead
        // (every thread reads the same table entry).  Otherwise the threads build the tile's row and
        // column offset arrays in shared memory, one entry each, also fetched one tile ahead.
        const bool regular = p.skinny_regular != 0;
        SkinnyWork w = skinny_work_at(p, t0);
        int64_t next_row = 0, next_col = 0;
        auto fetch = [&](const SkinnyWork &wk) {
            const int r = regular ? 0 : pt;
            next_row = r < wk.rows_valid ? p.offA_m[wk.m0 + r] + p.offA_h[wk.h] : 0;
            next_col = r < wk.cols_valid ? p.offB_n[wk.n0 + r] + p.offB_h[wk.h] : 0;
        };
        if (t0 < t1) fetch(w);
        BTC_PHASE_BEGIN();
#pragma unroll 1
        for (int64_t t = t0; t < t1; ++t) {
            const int i = int(t - t0), s = i & 1;
            const bool new_strip = t == t0 || w.nt == 0;
            if (new_strip) ++sidx;
            const int r = i % T::RAW_STAGES;
            int64_t *rA = rowA + (sidx & 1) * T::BM, *cB = colB + r * T::BN;
            const int64_t row_base = next_row, col_base = next_col;
            if (!regular) {
                if (new_strip) rA[pt] = next_row;
                cB[pt] = next_col;
                if (!umma_group_sync(loader_sync, unsigned(i) & 1u, abort_flag, p.error_word, p.poll_limit)) break;
            }
            const SkinnyWork wn = skinny_work_next(p, w);
            if (t + 1 < t1) fetch(wn);
            if (new_strip) {
                if (sidx > 0 && !mbar_wait_bounded(a_empty, unsigned(sidx - 1) & 1u, abort_flag, p.error_word, kErrSkinnyLoad, p.poll_limit)) break;
                if (regular) skinny_load_tile_regular<true>(araw, A, row_base, pieceA, pieces, p.dirA, w.rows_valid, pt, p.spans, 0);
                else skinny_load_tile<true>(araw, A, rA, koffA, pieceA, pieces, p.dirA, w.rows_valid, pt, p.spans, 0);
                mbar_arrive_on_copies(a_full);
            }
            BTC_PHASE_END(t_work);
            if (i >= T::RAW_STAGES &&
                !mbar_wait_bounded(raw_empty0 + 8u * r, unsigned(i / T::RAW_STAGES - 1) & 1u, abort_flag, p.error_word, kErrSkinnyLoad, p.poll_limit)) break;
            BTC_PHASE_END(t_wait);
            BTC_EVENT(p, pt == 0, 0, i);
            if (regular) skinny_load_tile_regular<false>(braw0 + unsigned(r) * T::B_BYTES, B, col_base, pieceB, pieces, p.dirB, w.cols_valid, pt, p.spans, 1);
            else skinny_load_tile<false>(braw0 + unsigned(r) * T::B_BYTES, B, cB, koffB, pieceB, pieces, p.dirB, w.cols_valid, pt, p.spans, 1);
            mbar_arrive_on_copies(raw_full0 + 8u * r);
            BTC_EVENT(p, pt == 0, 1, i);
            w = wn;
        }
        BTC_PHASE_END(t_work);
        BTC_PHASE_STORE(p, pt == 0, 4, t_wait);
        BTC_PHASE_STORE(p, pt == 0, 5, t_work);
        cp_async_wait_all();
    } else {
        // ------------------------------------------------------------- MMA warp
        constexpr unsigned IDESC_KK = umma_instr_desc(T::BN, false, false);
        constexpr unsigned IDESC_KM = umma_instr_desc(T::BN, false, true);
        const bool b_mn = p.dirB == 0;
        const unsigned idesc = b_mn ? IDESC_KM : IDESC_KK;       // the operand in tensor memory is K-major
        const unsigned b_lay = b_mn ? 1u : 2u, b_lbo = b_mn ? 512u : 16u, b_sbo = b_mn ? 16u * T::BN : 1024u;
        const unsigned b_step = b_mn ? 32u * T::BN : 32u;        // 8 k: two k-atoms, or 32 bytes of a row
        const bool leader = elect_one();
        int sidx = -1;
        long long t_acc = 0, t_conv = 0, t_issue = 0;
        (void)t_acc; (void)t_conv; (void)t_issue;
        int nt = skinny_work_at(p, t0).nt;
        BTC_PHASE_BEGIN();
#pragma unroll 1
        for (int64_t t = t0; t < t1; ++t) {
            const int i = int(t - t0), s = i & 1, buf = i & 1;
            const bool new_strip = t == t0 || nt == 0;
            if (++nt == p.tiles_n) nt = 0;           // now the column of the next tile
            if (new_strip) {
                ++sidx;
                if (!mbar_wait_bounded(ta_full0 + 8u * (sidx & 1), unsigned(sidx >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            }
            BTC_PHASE_END(t_issue);
            if (i >= 2 && !mbar_wait_bounded(acc_empty0 + 8u * buf, unsigned((i >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            BTC_PHASE_END(t_acc);
            if (!mbar_wait_bounded(lo_conv0 + 8u * s, unsigned(i >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            BTC_PHASE_END(t_conv);
            BTC_EVENT(p, lane == 0, 4, i);
            tc_fence_after();
            if (leader) {
                const unsigned tacc = tmem_base + unsigned(buf * T::ACC_COLS);
                const unsigned ta = tmem_a0 + unsigned((sidx & 1) * T::A_COLS);      // head columns; tail KMAX further
                const unsigned b_hi = braw0 + unsigned(i % T::RAW_STAGES) * T::B_BYTES, b_lo = blo0 + unsigned(s) * T::B_BYTES;
#pragma unroll 1
                for (int j = 0; j < ksteps; ++j) {
                    const unsigned at = unsigned(j >> 2) * T::B_BLOCK_BYTES + unsigned(j & 3) * b_step;
                    const uint64_t dbh = umma_smem_desc(b_hi + at, b_lbo, b_sbo, b_lay);
                    const uint64_t dbl = umma_smem_desc(b_lo + at, b_lbo, b_sbo, b_lay);
                    umma_tf32_ts(tacc, ta + unsigned(T::KMAX + 8 * j), dbh, idesc, j > 0 ? 1u : 0u);
                    umma_tf32_ts(tacc, ta + unsigned(8 * j), dbl, idesc, 1u);
                    umma_tf32_ts(tacc, ta + unsigned(8 * j), dbh, idesc, 1u);
                }
                umma_commit(raw_empty0 + 8u * unsigned(i % T::RAW_STAGES));       // fire when these MMAs have read the stages
                umma_commit(lo_empty0 + 8u * s);
                umma_commit(acc_full0 + 8u * buf);
                if (t + 1 == t1 || nt == 0) umma_commit(ta_empty0 + 8u * (sidx & 1));
            }
            __syncwarp();
            BTC_EVENT(p, lane == 0, 5, i);
        }
        BTC_PHASE_STORE(p, lane == 0, 6, t_acc);
        BTC_PHASE_STORE(p, lane == 0, 7, t_conv);
        tc_fence_before();
    }

    // ---- common tail: every role arrives here, also after an abort ----
    __syncthreads();
    if (warp == T::MMA_WARP) {
        if (*abort_flag) {
            // after an abort MMAs may still be running: wait (bounded) until the tensor core has drained
            if (elect_one()) umma_commit(drain);
            __syncwarp();
            for (unsigned n = 0; n < (1u << 16) && !mbar_try_wait(drain, 0u); ++n) { }
        }
        tc_fence_after();
        tmem_dealloc(tmem_base, T::TMEM_COLS);
    }
}

}  // namespace btc

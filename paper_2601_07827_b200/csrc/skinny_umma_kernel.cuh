// Bandwidth-bound fp32 contraction for short contracted extents (K <= 64) on the 5th-generation
// tensor cores: the low-intensity path of the contraction D = alpha op(A) op(B) + beta op(C)
// (Eq. (case2)) for shapes such as tensor-network contractions of many small modes, where the
// result is far larger than the inputs and the kernel's job is to stream D at memory speed.
//
// All of K fits one shared-memory tile, so there is no k loop and no stage ring along k.
// Persistent CTAs (one per SM) each take a contiguous range of the 128 x 128 output tiles, ordered
// (batch entry, pair of tile rows, tile column, half of the pair): the tiles of one tile row share their
// M-side operand tile ("strip"), which is fetched and converted once per strip and stays in tensor
// memory, and the two tiles of a pair share their N-side tile, so every operand tile fetched feeds two
// output tiles (a 256 x 128 block of D per 128 x K tile of B).
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
    // the N-side tiles wait in a ring of raw stages (each serves the two tiles of a pair, so two stages are
    // four tiles of lead over the tensor core); their tails are made just in time into a ring of the same
    // length; the M-side tile has two raw buffers, so that both halves' tiles of the next strip are
    // fetched while the tensor core still works on this one
    static constexpr int RAW_STAGES = 2, LO_STAGES = 2, A_STAGES = 2;
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
    static constexpr size_t SMEM_BYTES = size_t(RAW_STAGES + LO_STAGES) * B_BYTES + size_t(A_STAGES) * A_BYTES +
                                         size_t(2 * BM + RAW_STAGES * BN + 2 * KMAX) * 8 + size_t(2 * PIECES) * 4 +
                                         size_t(NUM_BARS) * 8 + 16 + 1024;
};

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

// A CTA's walk through its output tiles.  The tile list is ordered (batch entry, pair of tile rows, tile
// column, half of the pair) with the half fastest: the two tiles of a pair use the same N-side tile, which
// is therefore fetched and converted once for both (each half has its own M-side operand in tensor
// memory, kept for the whole strip).  With one tile row, or too few pairs to occupy the grid, halves = 1
// and every tile is its own pair.  A pair's second half may not exist (odd number of tile rows): the walk
// skips it.  Every role steps through the same walk, so the counters below agree between them.
struct SkinnyIter {
    int64_t h, left;         // batch entry; slots from this one to the end of the CTA's range
    int halves, half, nt, mt, since;
    int i, bi, an0, an1;     // tiles before this one; N-side tiles before this one's; M-side tiles loaded before, per half
    int abuf;                // tensor-memory buffer of this tile's M-side operand: its half, or (halves = 1) alternating by strip
    bool valid, new_a;       // new_a: the first tile of its half's strip for this CTA (its M-side tile must be loaded)

    __device__ __forceinline__ void start(const TiledParams &p, int halves_, int64_t pair0, int64_t pair1)
    {
        halves = halves_;
        const int tiles_mp = (p.tiles_m + halves - 1) / halves;
        nt = int(pair0 % p.tiles_n);
        const int64_t q = pair0 / p.tiles_n;
        mt = int(q % tiles_mp) * halves;
        h = q / tiles_mp;
        half = 0; since = 0;
        left = (pair1 - pair0) * halves;
        valid = left > 0;
        i = bi = an0 = an1 = abuf = 0;
        new_a = true;
    }
    __device__ __forceinline__ void advance(const TiledParams &p)
    {
        if (new_a) { if (half) ++an1; else ++an0; }
        for (;;) {
            --left; ++since;
            if (left <= 0) { valid = false; return; }
            if (++half == halves) {
                half = 0;
                mt -= halves - 1;
                if (++nt == p.tiles_n) {
                    nt = 0;
                    mt += halves;
                    if (mt >= p.tiles_m) { mt = 0; ++h; }
                }
            } else {
                ++mt;
            }
            if (mt < p.tiles_m) break;
        }
        ++i;
        if (half == 0) ++bi;
        new_a = nt == 0 || since < halves;
        if (halves == 2) abuf = half;
        else if (new_a) abuf = an0 & 1;
    }
    __device__ __forceinline__ bool first_of_b() const { return half == 0; }
    __device__ __forceinline__ bool last_of_b(const TiledParams &p) const { return half == halves - 1 || mt + 1 >= p.tiles_m; }
    // no later tile of this CTA uses this half's M-side operand
    __device__ __forceinline__ bool last_for_a(const TiledParams &p) const { return nt + 1 == p.tiles_n || left <= halves; }
    // at a tile with new_a: how often this tile's operand buffer has been filled before
    __device__ __forceinline__ int a_before() const { return halves == 1 ? (an0 >> 1) : (half ? an1 : an0); }
    __device__ __forceinline__ SkinnyWork work(const TiledParams &p) const
    {
        SkinnyWork w;
        w.h = h; w.mt = mt; w.nt = nt;
        w.m0 = int64_t(mt) * SkinnyTile::BM;
        w.n0 = int64_t(nt) * SkinnyTile::BN;
        w.rows_valid = int(imin64(SkinnyTile::BM, p.M - w.m0));
        w.cols_valid = int(imin64(SkinnyTile::BN, p.N - w.n0));
        return w;
    }
};

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
    int64_t ro0, ro1, ro_next, co_next[4];           // row offsets of the two halves' strips
    bool ok0, ok1, row_ok_next;

    __device__ __forceinline__ void init(const TiledParams &p, int row_, int lane_)
    {
        D = static_cast<float *>(p.D);
        C = static_cast<const float *>(p.C);
        alpha = float(p.alpha[0]); beta = float(p.beta[0]);
        vecn = p.skinny_vec_n == 4; dreg = p.skinny_d_regular != 0;
        row = row_; lane = lane_;
        ro0 = ro1 = ro_next = 0; ok0 = ok1 = row_ok_next = false;
        co_next[0] = co_next[1] = co_next[2] = co_next[3] = 0;
    }
    // start fetching what tile wk needs; `strip_start`: wk is the first tile of its half's strip for this CTA
    __device__ __forceinline__ void fetch(const TiledParams &p, const SkinnyBatch &sb, const SkinnyWork &wk, bool strip_start)
    {
        if (strip_start) {
            row_ok_next = row < wk.rows_valid;
            ro_next = row_ok_next ? p.offD_m[wk.m0 + row] + (sb.count ? sb.offD_h[wk.h] : p.offD_h[wk.h]) : 0;
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
    // the strip of half `half` starts: what fetch() brought is its row offset
    __device__ __forceinline__ void take_rows(int half)
    {
        if (half) { ro1 = ro_next; ok1 = row_ok_next; } else { ro0 = ro_next; ok0 = row_ok_next; }
    }
    // Columns [c_begin, c_end) (multiples of 32) of the accumulator at `tacc` (this warp's lane quarter)
    // -> D.  `co` = the column offsets fetched for this tile.  Arrives on `done_bar` as soon as the
    // columns are in registers.
    __device__ __forceinline__ void tile(const TiledParams &p, const SkinnyWork &w, int half, unsigned tacc, int c_begin, int c_end,
                                         unsigned done_bar, const int64_t (&co)[4])
    {
        const int64_t ro = half ? ro1 : ro0;
        const bool row_ok = half ? ok1 : ok0;
        const bool lean = vecn && dreg && !p.use_c && w.rows_valid == SkinnyTile::BM && w.cols_valid == SkinnyTile::BN;
        (void)lean;
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
#ifndef BTC_CHECK_OFFSETS
            if (lean) {
                // whole tile, regular columns, no C: nothing to decide per store
                float *base = D + (ro + co[0]);
                if (alpha == 1.f) {                  // the accumulator registers go out as they are
#pragma unroll
                    for (int q = 0; q < 8; ++q)
                        *reinterpret_cast<uint4 *>(base + p.skinny_col_rel[c0 + 4 * q]) = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
                    continue;
                }
#pragma unroll
                for (int q = 0; q < 8; ++q)
                    *reinterpret_cast<float4 *>(base + p.skinny_col_rel[c0 + 4 * q]) =
                        make_float4(alpha * __uint_as_float(r[4 * q]), alpha * __uint_as_float(r[4 * q + 1]),
                                    alpha * __uint_as_float(r[4 * q + 2]), alpha * __uint_as_float(r[4 * q + 3]));
                continue;
            }
#endif
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

__global__ void __launch_bounds__(SkinnyTile::THREADS, 1) skinny_umma_kernel(const __grid_constant__ TiledParams p, const __grid_constant__ SkinnyBatch sb)
{
    using T = SkinnyTile;
    extern __shared__ __align__(16) unsigned char smem_unaligned[];
    unsigned char *smem_raw = smem_unaligned +
        ((1024u - (static_cast<unsigned>(__cvta_generic_to_shared(smem_unaligned)) & 1023u)) & 1023u);
    unsigned char *cursor = smem_raw + size_t(T::RAW_STAGES + T::LO_STAGES) * T::B_BYTES + size_t(T::A_STAGES) * T::A_BYTES;
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
    const unsigned araw0 = blo0 + unsigned(T::LO_STAGES) * T::B_BYTES;      // two raw M-side buffers
    const unsigned bar0 = static_cast<unsigned>(__cvta_generic_to_shared(bars));
    const unsigned a_full0 = bar0, a_empty0 = bar0 + 16u;                                     // [2] each
    const unsigned raw_full0 = bar0 + 32u, raw_empty0 = raw_full0 + 8u * T::RAW_STAGES;       // [RAW_STAGES] each
    const unsigned lo_conv0 = raw_empty0 + 8u * T::RAW_STAGES, lo_empty0 = lo_conv0 + 16u;    // [2] each
    const unsigned ta_full0 = lo_empty0 + 16u, ta_empty0 = ta_full0 + 16u;                    // [2] each
    const unsigned acc_full0 = ta_empty0 + 16u, acc_empty0 = acc_full0 + 16u;                 // [2] each
    const unsigned loader_sync = acc_empty0 + 16u, drain = loader_sync + 8u;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int K = int(p.K);
    const int ksteps = (K + 7) / 8, kp = 8 * ksteps;                     // tensor-core steps of 8 k; k padded with zeros
    const int pieces = 32 * kp;                                         // 16-byte pieces of an operand tile in use
    // pairs of tile rows share their N-side tiles when that leaves a pair or more for every CTA
    const int halves = (p.tiles_m >= 2 && int64_t((p.tiles_m + 1) / 2) * p.tiles_n * p.Bt >= int64_t(gridDim.x)) ? 2 : 1;
    const int64_t total = int64_t((p.tiles_m + halves - 1) / halves) * p.tiles_n * p.Bt;      // pairs
    const int64_t t0 = total * blockIdx.x / gridDim.x, t1 = total * (blockIdx.x + 1) / gridDim.x;

    // the next grid in the stream may begin its own set-up as soon as SMs become free
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // ---- set-up: k offsets, barriers, tensor memory ----
    for (int i = tid; i < T::KMAX; i += T::THREADS) {
        koffA[i] = i < K ? p.offA_k[i] : 0;
        koffB[i] = i < K ? p.offB_k[i] : 0;
    }
    for (int e = tid; e < pieces; e += T::THREADS) {      // the piece tables, as the host prepared them
        pieceA[e] = p.skinny_orderA[e];
        pieceB[e] = p.skinny_orderB[e];
    }
    if (tid == 0) {
        for (int s = 0; s < 2; ++s) {
            mbar_init(a_full0 + 8u * s, T::GROUP_THREADS);
            mbar_init(a_empty0 + 8u * s, T::GROUP_THREADS);
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
    // Up to here only the operation's own tables were read.  From here on operand data is read and D is
    // written: the grid launched before this one in the stream must be complete and its writes visible.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const unsigned tmem_a0 = tmem_base + 2u * T::ACC_COLS;

    if (warp < T::EPILOGUE_WARPS) {
        // ------------------------------------------------------------- epilogue (first half of the columns)
        SkinnyStore st;
        st.init(p, tid, lane);
        SkinnyIter it;
        it.start(p, halves, t0, t1);
        if (it.valid) st.fetch(p, sb, it.work(p), true);
#pragma unroll 1
        while (it.valid) {
            const int i = it.i, buf = i & 1, half = it.half;
            const SkinnyWork w = it.work(p);
            if (it.new_a) st.take_rows(half);
            int64_t co[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) co[c] = st.co_next[c];
            it.advance(p);
            if (it.valid) st.fetch(p, sb, it.work(p), it.new_a);
            if (!mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(i >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit)) break;
            tc_fence_after();
            st.tile(p, w, half, tmem_base + (unsigned(warp * 32) << 16) + unsigned(buf * T::ACC_COLS), 0, T::SPLIT_COL, acc_empty0 + 8u * buf, co);
        }
    } else if (warp < T::EPILOGUE_WARPS + T::CONVERTER_WARPS) {
        // ------------------------------------------------------------- converters
        const int ct = tid - 32 * T::EPILOGUE_WARPS;             // row of the M-side tile = tensor-memory lane
        // Between conversions these warps also write the second half of the columns of the tile before
        // (its accumulator is complete by then), which doubles the warps that keep stores in flight.
        SkinnyStore st;
        st.init(p, ct, lane);
        SkinnyIter it;
        it.start(p, halves, t0, t1);
        SkinnyWork wprev = it.work(p);
        int half_prev = 0, i_last = -1;
        int64_t co_prev[4] = {0, 0, 0, 0};
        bool ok = true;
#pragma unroll 1
        while (it.valid) {
            const int i = it.i, half_now = it.half;
            const SkinnyWork w = it.work(p);
            const bool new_a = it.new_a;
            st.fetch(p, sb, w, new_a);                    // for this tile's store, one iteration from now
            if (new_a) {
                const int loads = it.an0 + it.an1, mine = it.a_before(), ab = it.abuf;
                const unsigned araw = araw0 + unsigned(loads & 1) * T::A_BYTES;
                if (!(ok = mbar_wait_bounded(a_full0 + 8u * unsigned(loads & 1), unsigned(loads >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit))) break;
                // the operand buffer is free once the tensor core has finished the strip that used it before
                if (mine >= 1 &&
                    !(ok = mbar_wait_bounded(ta_empty0 + 8u * ab, unsigned(mine - 1) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit)))
                    break;
                tc_fence_after();
                const unsigned ta = tmem_a0 + unsigned(ab * T::A_COLS) + (unsigned(ct & ~31) << 16);
#pragma unroll
                for (int kh = 0; kh < 2; ++kh) {
                    if (kh * 32 >= kp) break;
                    float x[32];
                    if (p.dirA == 0) {
#pragma unroll
                        for (int k = 0; k < 32; ++k)
                            asm volatile("ld.shared.f32 %0, [%1];" : "=f"(x[k]) : "r"(araw + unsigned((kh * 32 + k) * T::BM + ct) * 4u) : "memory");
                    } else {
#pragma unroll
                        for (int c = 0; c < 8; ++c)
                            asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                                         : "=f"(x[4 * c]), "=f"(x[4 * c + 1]), "=f"(x[4 * c + 2]), "=f"(x[4 * c + 3])
                                         : "r"(araw + unsigned(ct) * 256u + (unsigned(((kh * 8 + c) ^ ct) & 15) << 4)) : "memory");
                    }
                    tmem_store32(ta + unsigned(kh * 32), x);
#pragma unroll
                    for (int k = 0; k < 32; ++k) x[k] -= __uint_as_float(__float_as_uint(x[k]) & 0xffffe000u);
                    tmem_store32(ta + unsigned(T::KMAX + kh * 32), x);
                }
                tmem_store_wait();
                tc_fence_before();
                mbar_arrive(ta_full0 + 8u * ab);
                mbar_arrive(a_empty0 + 8u * unsigned(loads & 1));     // this raw M-side buffer may be refilled
            }
            if (it.first_of_b()) {
                const int bi = it.bi, r = bi % T::RAW_STAGES, s = bi & 1;
                if (!(ok = mbar_wait_bounded(raw_full0 + 8u * r, unsigned(bi / T::RAW_STAGES) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit))) break;
                // the tail stage is free once the tensor core has finished the tiles of the N-side tile two before
                if (bi >= 2 && !(ok = mbar_wait_bounded(lo_empty0 + 8u * s, unsigned((bi >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyConvert, p.poll_limit))) break;
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
                proxy_fence_async();                  // the tensor core reads both stages through the async proxy
                mbar_arrive(lo_conv0 + 8u * s);
            }
            if (i > 0) {
                const int ip = i - 1, buf = ip & 1;
                if (!(ok = mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(ip >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit))) break;
                tc_fence_after();
                st.tile(p, wprev, half_prev, tmem_base + (unsigned(ct & ~31) << 16) + unsigned(buf * T::ACC_COLS), T::SPLIT_COL, T::BN,
                        acc_empty0 + 8u * buf, co_prev);
            }
            // what was fetched at the top of this iteration belongs to this tile: keep it for the next iteration
#pragma unroll
            for (int c = 0; c < 4; ++c) co_prev[c] = st.co_next[c];
            if (new_a) st.take_rows(half_now);
            wprev = w; half_prev = half_now; i_last = i;
            it.advance(p);
        }
        if (ok && i_last >= 0 && !*abort_flag) {      // the last tile's second half of the columns
            const int buf = i_last & 1;
            if (mbar_wait_bounded(acc_full0 + 8u * buf, unsigned(i_last >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyEpilogue, p.poll_limit)) {
                tc_fence_after();
                st.tile(p, wprev, half_prev, tmem_base + (unsigned(ct & ~31) << 16) + unsigned(buf * T::ACC_COLS), T::SPLIT_COL, T::BN,
                        acc_empty0 + 8u * buf, co_prev);
            }
        }
    } else if (warp < T::MMA_WARP) {
        // ------------------------------------------------------------- loaders
        const int pt = tid - 32 * (T::EPILOGUE_WARPS + T::CONVERTER_WARPS);
        const float *A = static_cast<const float *>(p.A), *B = static_cast<const float *>(p.B);
        // Regular operands: a tile is addressed by its first row's offset alone, fetched one tile ahead
        // (every thread reads the same table entry).  Otherwise the threads build the tile's row and
        // column offset arrays in shared memory, one entry each, also fetched one tile ahead.
        const bool regular = p.skinny_regular != 0;
        SkinnyIter it;
        it.start(p, halves, t0, t1);
        int64_t next_row = 0, next_col = 0;
        auto fetch = [&](const SkinnyIter &at) {
            const SkinnyWork wk = at.work(p);
            const int r = regular ? 0 : pt;
            if (at.new_a) next_row = r < wk.rows_valid ? p.offA_m[wk.m0 + r] + (sb.count ? sb.offA_h[wk.h] : p.offA_h[wk.h]) : 0;
            if (at.first_of_b()) next_col = r < wk.cols_valid ? p.offB_n[wk.n0 + r] + (sb.count ? sb.offB_h[wk.h] : p.offB_h[wk.h]) : 0;
        };
        if (it.valid) fetch(it);
#pragma unroll 1
        while (it.valid) {
            const int i = it.i, bi = it.bi, r = bi % T::RAW_STAGES, loads = it.an0 + it.an1;
            const bool new_a = it.new_a, new_b = it.first_of_b();
            const SkinnyWork w = it.work(p);
            int64_t *rA = rowA + (loads & 1) * T::BM, *cB = colB + r * T::BN;
            const int64_t row_base = next_row, col_base = next_col;
            if (!regular) {
                if (new_a) rA[pt] = next_row;
                if (new_b) cB[pt] = next_col;
                if (!umma_group_sync(loader_sync, unsigned(i) & 1u, abort_flag, p.error_word, p.poll_limit)) break;
            }
            it.advance(p);
            if (it.valid) fetch(it);
            if (new_a) {
                const unsigned araw = araw0 + unsigned(loads & 1) * T::A_BYTES;
                if (loads >= 2 &&
                    !mbar_wait_bounded(a_empty0 + 8u * unsigned(loads & 1), unsigned((loads >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyLoad, p.poll_limit)) break;
                if (regular) skinny_load_tile_regular<true>(araw, A, row_base, pieceA, pieces, p.dirA, w.rows_valid, pt, p.spans, 0);
                else skinny_load_tile<true>(araw, A, rA, koffA, pieceA, pieces, p.dirA, w.rows_valid, pt, p.spans, 0);
                mbar_arrive_on_copies(a_full0 + 8u * unsigned(loads & 1));
            }
            if (new_b) {
                if (bi >= T::RAW_STAGES &&
                    !mbar_wait_bounded(raw_empty0 + 8u * r, unsigned(bi / T::RAW_STAGES - 1) & 1u, abort_flag, p.error_word, kErrSkinnyLoad, p.poll_limit)) break;
                if (regular) skinny_load_tile_regular<false>(braw0 + unsigned(r) * T::B_BYTES, B, col_base, pieceB, pieces, p.dirB, w.cols_valid, pt, p.spans, 1);
                else skinny_load_tile<false>(braw0 + unsigned(r) * T::B_BYTES, B, cB, koffB, pieceB, pieces, p.dirB, w.cols_valid, pt, p.spans, 1);
                mbar_arrive_on_copies(raw_full0 + 8u * r);
            }
        }
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
        SkinnyIter it;
        it.start(p, halves, t0, t1);
#pragma unroll 1
        for (; it.valid; it.advance(p)) {
            const int i = it.i, buf = i & 1, bi = it.bi, r = bi % T::RAW_STAGES, s = bi & 1;
            if (it.new_a &&
                !mbar_wait_bounded(ta_full0 + 8u * unsigned(it.abuf), unsigned(it.a_before()) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            if (i >= 2 && !mbar_wait_bounded(acc_empty0 + 8u * buf, unsigned((i >> 1) - 1) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            if (it.first_of_b() &&
                !mbar_wait_bounded(lo_conv0 + 8u * s, unsigned(bi >> 1) & 1u, abort_flag, p.error_word, kErrSkinnyMma, p.poll_limit)) break;
            tc_fence_after();
            if (leader) {
                const unsigned tacc = tmem_base + unsigned(buf * T::ACC_COLS);
                const unsigned ta = tmem_a0 + unsigned(it.abuf * T::A_COLS);            // head columns; tail KMAX further
                const unsigned b_hi = braw0 + unsigned(r) * T::B_BYTES, b_lo = blo0 + unsigned(s) * T::B_BYTES;
#pragma unroll 1
                for (int j = 0; j < ksteps; ++j) {
                    const unsigned at = unsigned(j >> 2) * T::B_BLOCK_BYTES + unsigned(j & 3) * b_step;
                    const uint64_t dbh = umma_smem_desc(b_hi + at, b_lbo, b_sbo, b_lay);
                    const uint64_t dbl = umma_smem_desc(b_lo + at, b_lbo, b_sbo, b_lay);
                    umma_tf32_ts(tacc, ta + unsigned(T::KMAX + 8 * j), dbh, idesc, j > 0 ? 1u : 0u);
                    umma_tf32_ts(tacc, ta + unsigned(8 * j), dbl, idesc, 1u);
                    umma_tf32_ts(tacc, ta + unsigned(8 * j), dbh, idesc, 1u);
                }
                if (it.last_of_b(p)) {                // fire when the MMAs so far have read the stages
                    umma_commit(raw_empty0 + 8u * unsigned(r));
                    umma_commit(lo_empty0 + 8u * s);
                }
                umma_commit(acc_full0 + 8u * buf);
                if (it.last_for_a(p)) umma_commit(ta_empty0 + 8u * unsigned(it.abuf));
            }
            __syncwarp();
        }
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

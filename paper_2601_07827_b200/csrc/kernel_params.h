// Parameter blocks shared by the host launchers and the device kernels.
#pragma once

#include <cstdint>

namespace btc {

// Memory span of each tensor in elements relative to its pointer ([lo, hi] inclusive; 0: M-side input,
// 1: N-side input, 2: D and C) and the device error word.  Debug builds (-DBTC_CHECK_OFFSETS) compare every
// global offset the kernels compute with these and record kErrOffsetRange instead of making the access.
struct OffsetSpans {
    int64_t lo[3], hi[3];
    int32_t *error_word;
};
constexpr int kErrOffsetRange = 20;

#if defined(BTC_CHECK_OFFSETS) && defined(__CUDACC__)
__device__ __forceinline__ bool offset_in_span(const OffsetSpans &s, int which, int64_t off, int count)
{
    const bool ok = off >= s.lo[which] && off + count - 1 <= s.hi[which];
    if (!ok && s.error_word) atomicCAS(s.error_word, 0, kErrOffsetRange);
    return ok;
}
#define BTC_IN_SPAN(spans, which, off, count) offset_in_span(spans, which, off, count)
#else
#define BTC_IN_SPAN(spans, which, off, count) true
#endif

constexpr int kGenericMaxD = 32;   // loop dimensions over D (batch + free), after merging
constexpr int kGenericMaxK = 64;   // summed loop dimensions

// One thread (or one warp) per element of D; used for every input the tiled kernels decline.
struct GenericParams {
    const void *A, *B, *C;
    void *D;
    int32_t nd, nk;
    int64_t total_d, total_k;
    int64_t ext_d[kGenericMaxD], sA_d[kGenericMaxD], sB_d[kGenericMaxD], sD_d[kGenericMaxD];
    int64_t ext_k[kGenericMaxK], sA_k[kGenericMaxK], sB_k[kGenericMaxK];
    double alpha[2], beta[2];
    int32_t conjA, conjB, conjC;
    int32_t use_ab, use_c;
    int32_t cplxA, cplxB, cplxC;      // 1: that operand's elements are (re, im) pairs; D's type is the kernel's
    OffsetSpans spans;
};

// Sum over the isolated labels of one input (Case 4): kept and isolated loop dimensions of the
// tensor, each with its extent and element stride, first entry fastest.
struct IsolatedSumParams {
    const void *src;
    void *dst;                        // dense, kept dimensions in the order given here
    int32_t nk, ni;
    int64_t total_keep, total_iso;
    int64_t ext_k[kGenericMaxD], str_k[kGenericMaxD], ext_i[kGenericMaxD], str_i[kGenericMaxD];
};

// C := alpha op(A) + beta op(B): loop dimensions over C (extent, element strides in A, B, C; A's
// stride is 0 where A is broadcast), first entry fastest, and the dimensions summed over in A.
struct ElementwiseParams {
    const void *A, *B;
    void *C;
    int32_t nk, ns;
    int64_t total_keep, total_sum;
    int64_t ext_k[kGenericMaxD], sA_k[kGenericMaxD], sB_k[kGenericMaxD], sC_k[kGenericMaxD];
    int64_t ext_s[kGenericMaxD], sA_s[kGenericMaxD];
    // division by ext_k[d] (and by ext_k[0] / vector length, last entry) without a divide, for 32-bit
    // indices below 2^31: q = (n * div_mul) >> div_shift in 64 bits, div_shift = 31 + ceil(log2 ext),
    // div_mul = ceil(2^div_shift / ext) (exact for n < 2^31 since div_mul * ext - 2^div_shift < ext)
    uint32_t div_mul[kGenericMaxD + 1], div_shift[kGenericMaxD + 1];
    int32_t tile_mode_a;              // transposing kernel: the dimension A is read along (C: dimension 0)
    int32_t tiles_c, tiles_a;         // transposing kernel: tiles along those two dimensions
    int64_t rest;                     // transposing kernel: product of the other dimensions' extents
    double alpha[2], beta[2];
    int32_t conjA, conjB;
    int32_t use_a, use_b;
};

// Tiled contraction kernels.  All offsets are in elements of the operation's dtype.
struct TiledParams {
    const void *A, *B, *C;
    void *D;
    const int64_t *offA_m, *offD_m;   // [M]
    const int64_t *offB_n, *offD_n;   // [N]
    const int64_t *offA_k, *offB_k;   // [K]
    const int64_t *offA_h, *offB_h, *offD_h;   // [Bt]
    int64_t M, N, K, Bt;
    int32_t tiles_m, tiles_n;
    int32_t bm, bn;                   // CTA tile extents in elements
    int32_t raster_n_fast;            // 1: consecutive CTAs walk the n tiles of one m tile
    int32_t split_k;
    int64_t k_per_split;              // multiple of the K tile
    int32_t dirA, dirB;               // 0: threads run along the free index, 1: along k
    int32_t vecA, vecB;               // elements per global->shared copy
    int32_t vecD;                     // v > 1: groups of v consecutive m are v consecutive, 16-byte aligned elements of D
    int32_t conjA, conjB, conjC;
    int32_t use_c;
    double alpha[2], beta[2];
    void *partials;                   // split-K scratch (workspace), or nullptr
    // 1 (fp64 kernels, split_k = 2, 4 or 8): the CTAs of one tile's k slices form a thread-block cluster
    // (slice = rank in the cluster, so the work list runs slice-fastest) and add their partial tiles through
    // distributed shared memory: one launch, no scratch
    int32_t cluster_split;
    int32_t *error_word;              // device word; set non-zero when a bounded wait gave up
    uint32_t poll_limit;              // polls after which a device-side wait gives up
    OffsetSpans spans;                // what the offset checks of debug builds compare with
    // bulk-tensor-copy variants: box origin of the M-side operand = coord_m[tile of M] + coord_k[stage]
    // + coord_h[batch entry], five coordinates each
    const int32_t *tmaA_coord_m, *tmaA_coord_k, *tmaA_coord_h;
    // short-K streaming kernel: the 16-byte pieces of an operand tile (128 rows x up to 64 k), each
    // list sorted by address in its tensor (see skinny_umma_kernel.cuh); skinny_vec_n = 4: groups of
    // four consecutive n are four consecutive, 16-byte aligned elements of D (and C)
    const uint32_t *skinny_orderA, *skinny_orderB;
    int32_t skinny_vec_n;
    // 1: in both operands every tile's rows lie relative to the tile's first row as those of tile 0 do, and
    // the offsets inside a tile fit 32 bits: tiles are addressed by their first row's offset alone
    int32_t skinny_regular;
    // 1: D's columns are regular in the same sense; column c of a tile then lies skinny_col_rel[c] elements
    // after the tile's first column (read through the constant bank instead of per-lane tables)
    int32_t skinny_d_regular;
    int32_t skinny_col_rel[128];
};

// Short-K streaming kernel, pointer-array calls of few entries: the per-entry offsets ride in the kernel's
// parameters instead of a table uploaded before the launch (count = 0: the tables of TiledParams count).
constexpr int kSkinnyInlineEntries = 64;
struct SkinnyBatch {
    int32_t count, pad;
    int64_t offA_h[kSkinnyInlineEntries], offB_h[kSkinnyInlineEntries], offD_h[kSkinnyInlineEntries];
};

}  // namespace btc

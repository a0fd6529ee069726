// Building blocks shared by the tiled contraction kernels: asynchronous copies, mbarriers with
// bounded waits, register re-balancing between warpgroups, and the strided-tile gather that the
// producer warps run.
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

namespace btc {

constexpr int kProducerWarps = 4;   // one warpgroup

// k-offset entries per operand that a CTA keeps in shared memory (its whole k slice when it fits)
constexpr int kKoffCap = 1024;

__device__ __forceinline__ int64_t imin64(int64_t a, int64_t b) { return a < b ? a : b; }

// ---- asynchronous copies and mbarriers ---------------------------------------------------------
template <int BYTES>
__device__ __forceinline__ void cp_async_bytes(unsigned dst, const void *gsrc, bool valid)
{
    const int src = valid ? BYTES : 0;   // src-size 0 zero-fills the destination
    if (BYTES == 16)
        asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(gsrc), "r"(src) : "memory");
    else if (BYTES == 8)
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(gsrc), "r"(src) : "memory");
    else
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(dst), "l"(gsrc), "r"(src) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

__device__ __forceinline__ void mbar_init(unsigned bar, int count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// the barrier receives one arrival from this thread once all its earlier cp.async have landed
__device__ __forceinline__ void mbar_arrive_on_copies(unsigned bar)
{
    asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity)
{
    unsigned ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
                 "selp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

constexpr unsigned kWaitPollLimit = 1u << 22;   // polls before a wait gives up (a poll itself blocks briefly)
constexpr int kErrFullWait = 1, kErrEmptyWait = 2, kErrSelfTest = 7;

// Bounded wait.  Returns false when it gave up or another warp raised the abort flag.
__device__ __forceinline__ bool mbar_wait_bounded(unsigned bar, unsigned parity, volatile int *abort_flag,
                                                  int *error_word, int code, unsigned poll_limit = kWaitPollLimit)
{
    for (unsigned n = 0; n < poll_limit; ++n) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((n & 255u) == 255u && *abort_flag) return false;
    }
    *abort_flag = 1;
    if (error_word) atomicCAS(error_word, 0, code);
    return false;
}

// Cluster-wide barrier of all threads that have not exited (release / acquire: shared-memory writes
// made before it are visible to the other CTAs of the cluster after it).
__device__ __forceinline__ void cluster_barrier()
{
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// the address of this CTA's shared-memory location `addr` in the CTA of rank `rank` of the cluster
__device__ __forceinline__ unsigned cluster_map(unsigned addr, unsigned rank)
{
    unsigned r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ double cluster_load_f64(unsigned addr)
{
    double v;
    asm volatile("ld.shared::cluster.f64 %0, [%1];" : "=d"(v) : "r"(addr) : "memory");
    return v;
}

// Self-test of the bounded wait: every thread waits on an mbarrier that nobody arrives on, with a
// small poll limit.  The wait must give up, raise the abort flag and write the error word; the
// kernel then returns normally, so the context stays usable.  (A template only so that the
// header can be included by several translation units.)
template <int UNUSED = 0>
__global__ void bounded_wait_selftest_kernel(unsigned poll_limit, int *error_word, int *gave_up_count)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ int abort_flag;
    const unsigned b = static_cast<unsigned>(__cvta_generic_to_shared(&bar));
    if (threadIdx.x == 0) {
        mbar_init(b, 1);
        abort_flag = 0;
    }
    __syncthreads();
    const bool done = mbar_wait_bounded(b, 0u, &abort_flag, error_word, kErrSelfTest, poll_limit);
    if (!done) atomicAdd(gave_up_count, 1);
}

template <int REGS> __device__ __forceinline__ void reg_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REGS)); }
template <int REGS> __device__ __forceinline__ void reg_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REGS)); }

// Gather one ROWS x BK tile (rows = free index, columns = k) into shared memory.
//   DIR       0: consecutive threads take consecutive rows; 1: consecutive k
//   VEC       elements per copy along that direction
//   row_off   shared array: element offset of each tile row (batch offset included)
//   koff      table of k offsets indexed by absolute k (global memory, or the CTA's shared copy
//             biased by the slice start);  [.., k_end) is this CTA's valid k range
//   s_row, s_k  shared-memory strides of the tile in elements
template <int ROWS, int BK, int NTHREADS, int ELEM_BYTES, int DIR, int VEC>
__device__ __forceinline__ void gather_tile(unsigned smem, const char *__restrict__ g, const int64_t *row_off,
                                            const int64_t *koff, int rows_valid, int64_t k0,
                                            int64_t k_end, int s_row, int s_k, int tid, const OffsetSpans &spans, int which)
{
    constexpr int NFAST = (DIR == 0 ? ROWS : BK) / VEC;
    constexpr int SLOTS = ROWS * BK / VEC;
    constexpr int PER = (SLOTS + NTHREADS - 1) / NTHREADS;     // copies per thread
    constexpr int BATCH = PER < 4 ? PER : 4;
    // offsets of a batch are looked up first and its copies issued together: a copy is an
    // ordered memory operation, so interleaving would serialise every table look-up behind it
#pragma unroll 1
    for (int base = 0; base < PER; base += BATCH) {
        int64_t off[BATCH];
        bool valid[BATCH];
#pragma unroll
        for (int j = 0; j < BATCH; ++j) {
            const int s = tid + (base + j) * NTHREADS;
            const int f = (s % NFAST) * VEC, o = s / NFAST;
            const int r = DIR == 0 ? f : o;
            const int k = DIR == 0 ? o : f;
            valid[j] = s < SLOTS && (r < rows_valid) && (k0 + k < k_end);
            off[j] = valid[j] ? row_off[r] + koff[k0 + k] : 0;
            if (valid[j] && !BTC_IN_SPAN(spans, which, off[j], VEC)) { valid[j] = false; off[j] = 0; }
        }
#pragma unroll
        for (int j = 0; j < BATCH; ++j) {
            const int s = tid + (base + j) * NTHREADS;
            if (s < SLOTS) {
                const int f = (s % NFAST) * VEC, o = s / NFAST;
                const int r = DIR == 0 ? f : o;
                const int k = DIR == 0 ? o : f;
                cp_async_bytes<VEC * ELEM_BYTES>(smem + unsigned(r * s_row + k * s_k) * ELEM_BYTES, g + off[j] * ELEM_BYTES, valid[j]);
            }
        }
    }
}

template <int ROWS, int BK, int NTHREADS, int ELEM_BYTES, int DIR>
__device__ __forceinline__ void gather_dispatch_vec(unsigned smem, const char *__restrict__ g, const int64_t *row_off,
                                                    const int64_t *koff, int rows_valid, int64_t k0,
                                                    int64_t k_end, int vec, int s_row, int s_k, int tid, const OffsetSpans &spans, int which)
{
    constexpr int VMAX = 16 / ELEM_BYTES;   // 4 for fp32, 2 for fp64 and complex64, 1 for complex128
    if (VMAX >= 4 && vec == 4)
        gather_tile<ROWS, BK, NTHREADS, ELEM_BYTES, DIR, (VMAX >= 4 ? 4 : 1)>(smem, g, row_off, koff, rows_valid, k0, k_end, s_row, s_k, tid, spans, which);
    else if (VMAX >= 2 && vec == 2)
        gather_tile<ROWS, BK, NTHREADS, ELEM_BYTES, DIR, (VMAX >= 2 ? 2 : 1)>(smem, g, row_off, koff, rows_valid, k0, k_end, s_row, s_k, tid, spans, which);
    else
        gather_tile<ROWS, BK, NTHREADS, ELEM_BYTES, DIR, 1>(smem, g, row_off, koff, rows_valid, k0, k_end, s_row, s_k, tid, spans, which);
}

template <int ROWS, int BK, int NTHREADS, int ELEM_BYTES>
__device__ __forceinline__ void gather_dispatch(unsigned smem, const char *__restrict__ g, const int64_t *row_off,
                                                const int64_t *koff, int rows_valid, int64_t k0,
                                                int64_t k_end, int dir, int vec, int s_row, int s_k, int tid, const OffsetSpans &spans, int which)
{
    if (dir == 0)
        gather_dispatch_vec<ROWS, BK, NTHREADS, ELEM_BYTES, 0>(smem, g, row_off, koff, rows_valid, k0, k_end, vec, s_row, s_k, tid, spans, which);
    else
        gather_dispatch_vec<ROWS, BK, NTHREADS, ELEM_BYTES, 1>(smem, g, row_off, koff, rows_valid, k0, k_end, vec, s_row, s_k, tid, spans, which);
}


// What every tiled kernel computes first: which tile / k slice / batch entry this CTA owns.
struct TileCoords {
    int tile, ks;
    int64_t h, m0, n0, k_begin, k_end;
    int rows_valid, cols_valid, num_kt;
};

// `work` enumerates (tile, k slice, batch), tile fastest -- or, where the slices of a tile form a
// cluster, (k slice, tile, batch), slice fastest
template <int BM, int BN, int BK, typename Params>
__device__ __forceinline__ TileCoords tile_coords_at(const Params &p, int64_t work)
{
    TileCoords c;
    const int tiles = p.tiles_m * p.tiles_n;
    c.tile = p.cluster_split ? int((work / p.split_k) % tiles) : int(work % tiles);
    c.ks = p.cluster_split ? int(work % p.split_k) : int((work / tiles) % p.split_k);
    c.h = work / (int64_t(tiles) * p.split_k);
    const int tile_m = p.raster_n_fast ? c.tile / p.tiles_n : c.tile % p.tiles_m;
    const int tile_n = p.raster_n_fast ? c.tile % p.tiles_n : c.tile / p.tiles_m;
    c.m0 = int64_t(tile_m) * BM;
    c.n0 = int64_t(tile_n) * BN;
    c.rows_valid = int(imin64(BM, p.M - c.m0));
    c.cols_valid = int(imin64(BN, p.N - c.n0));
    c.k_begin = int64_t(c.ks) * p.k_per_split;
    c.k_end = imin64(p.K, c.k_begin + p.k_per_split);
    c.num_kt = int((c.k_end - c.k_begin + BK - 1) / BK);
    return c;
}

// one CTA per work item
template <int BM, int BN, int BK, typename Params>
__device__ __forceinline__ TileCoords tile_coords(const Params &p)
{
    return tile_coords_at<BM, BN, BK>(p, int64_t(blockIdx.x));
}

// Per-tile row/column offset arrays (batch offset folded in) and the stage barriers; ends with a
// CTA-wide barrier.
template <int BM, int BN, int STAGES, int NTHREADS, int PRODUCERS, int CONSUMER_WARPS, typename Params>
__device__ __forceinline__ void tile_setup(const Params &p, const TileCoords &c, int64_t *rowA, int64_t *rowD,
                                           int64_t *colB, int64_t *colD, int64_t *koffA, int64_t *koffB,
                                           unsigned full0, unsigned empty0, volatile int *abort_flag, int tid)
{
    // the k offsets of this CTA's slice, when they fit: the producers then never wait on a
    // table load between a stage's release and its copies
    if (c.k_end - c.k_begin <= kKoffCap) {
        for (int i = tid; i < int(c.k_end - c.k_begin); i += NTHREADS) {
            koffA[i] = p.offA_k[c.k_begin + i];
            koffB[i] = p.offB_k[c.k_begin + i];
        }
    }
    const int64_t hA = p.offA_h[c.h], hB = p.offB_h[c.h], hD = p.offD_h[c.h];
    for (int i = tid; i < BM; i += NTHREADS) {
        const bool v = i < c.rows_valid;
        rowA[i] = v ? p.offA_m[c.m0 + i] + hA : 0;
        rowD[i] = v ? p.offD_m[c.m0 + i] + hD : 0;
    }
    for (int i = tid; i < BN; i += NTHREADS) {
        const bool v = i < c.cols_valid;
        colB[i] = v ? p.offB_n[c.n0 + i] + hB : 0;
        colD[i] = v ? p.offD_n[c.n0 + i] : 0;
    }
    if (tid == 0) {
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(full0 + 8u * s, PRODUCERS);
            mbar_init(empty0 + 8u * s, CONSUMER_WARPS);
        }
        *abort_flag = 0;
    }
    __syncthreads();
}

// The producer warpgroup's loop: wait until the consumers have released a stage, gather the next
// A and B tiles into it, and let the stage's "full" barrier fire when the copies have landed.
template <int BM, int BN, int BK, int EB, int STAGES, int STAGE_BYTES, int A_BYTES, int PRODUCERS, typename Params>
__device__ __forceinline__ void producer_loop(const Params &p, const TileCoords &c, unsigned stage0,
                                              const int64_t *rowA, const int64_t *colB, const int64_t *koffA,
                                              const int64_t *koffB, unsigned full0, unsigned empty0,
                                              volatile int *abort_flag, int a_srow, int a_sk, int b_srow, int b_sk,
                                              int tid)
{
    const bool staged = c.k_end - c.k_begin <= kKoffCap;
    const int64_t *ka = staged ? koffA - c.k_begin : p.offA_k;
    const int64_t *kb = staged ? koffB - c.k_begin : p.offB_k;
    for (int kt = 0; kt < c.num_kt; ++kt) {
        const int s = kt % STAGES, round = kt / STAGES;
        if (round > 0 &&
            !mbar_wait_bounded(empty0 + 8u * s, unsigned(round - 1) & 1u, abort_flag, p.error_word, kErrEmptyWait, p.poll_limit))
            break;
        const unsigned sa = stage0 + unsigned(s) * STAGE_BYTES;
        const unsigned sb = sa + A_BYTES;
        const int64_t k0 = c.k_begin + int64_t(kt) * BK;
        gather_dispatch<BM, BK, PRODUCERS, EB>(sa, static_cast<const char *>(p.A), rowA, ka, c.rows_valid, k0,
                                               c.k_end, p.dirA, p.vecA, a_srow, a_sk, tid, p.spans, 0);
        gather_dispatch<BN, BK, PRODUCERS, EB>(sb, static_cast<const char *>(p.B), colB, kb, c.cols_valid, k0,
                                               c.k_end, p.dirB, p.vecB, b_srow, b_sk, tid, p.spans, 1);
        mbar_arrive_on_copies(full0 + 8u * s);
    }
    cp_async_wait_all();
}

}  // namespace btc

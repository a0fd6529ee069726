// Epilogue shared by the tiled kernels:  D = alpha * acc + beta * op(C), written through D's
// offset tables (Eq. (case2): the alpha / beta step of the contraction).
//
// The consumer warps first park their accumulator fragments in shared memory as an image of
// the CTA tile, image[column][row] with rows contiguous (the stage buffers are free by then).
// All consumer threads then walk the image in one rolled loop, consecutive threads on
// consecutive rows, so that a D whose first M mode is contiguous is written in full, aligned
// 16-byte pieces, and the code executed once per CTA stays a few hundred instructions (a fully
// unrolled per-fragment epilogue costs microseconds of instruction fetch on small problems).
// With split-K the same walk writes the raw image to scratch, and one small kernel per element
// type adds the slices in a fixed order and applies alpha / beta.
#pragma once

#include <cuda_runtime.h>

#include "kernel_params.h"
#include "tile_common.cuh"

namespace btc {

// pitch (in elements) between image columns: rows + 4 keeps 16-byte alignment for every element
// type and spreads the fragment stores over the banks
template <int BM> struct ImagePitch { static constexpr int value = BM + 4; };

template <int THREADS> __device__ __forceinline__ void consumer_barrier()
{
    asm volatile("bar.sync 1, %0;" ::"n"(THREADS) : "memory");
}

// one element: acc -> alpha * acc + beta * op(c) -> D;  Acc = float or double, W = 1 (real) or 2;
// (c_r, c_i) is the element of C, already loaded (ignored when beta == 0)
template <typename Acc, int W>
__device__ __forceinline__ void finish_element(const TiledParams &p, int64_t off, Acc acc_r, Acc acc_i, Acc c_r, Acc c_i)
{
    Acc *D = static_cast<Acc *>(p.D);
    if (W == 2) {
        const Acc ar = Acc(p.alpha[0]), ai = Acc(p.alpha[1]);
        Acc d_r = ar * acc_r - ai * acc_i, d_i = ar * acc_i + ai * acc_r;
        if (p.use_c) {
            const Acc ci = p.conjC ? -c_i : c_i;
            const Acc br = Acc(p.beta[0]), bi = Acc(p.beta[1]);
            d_r += br * c_r - bi * ci;
            d_i += br * ci + bi * c_r;
        }
        D[2 * off] = d_r;
        D[2 * off + 1] = d_i;
    } else {
        Acc d = Acc(p.alpha[0]) * acc_r;
        if (p.use_c) d += Acc(p.beta[0]) * c_r;
        D[off] = d;
    }
}

// 16 bytes = V elements that are consecutive in the image, in C and in D
template <typename Acc, int W, int V> union Pack16 { uint4 raw; Acc w[V * W]; };

template <typename Acc, int W, int V>
__device__ __forceinline__ void finish_vector(const TiledParams &p, int64_t off, const Acc *image_words,
                                              const Pack16<Acc, W, V> &c)
{
    Pack16<Acc, W, V> a, d;
    a.raw = *reinterpret_cast<const uint4 *>(image_words);
    if (W == 2) {
        const Acc ar = Acc(p.alpha[0]), ai = Acc(p.alpha[1]), br = Acc(p.beta[0]), bi = Acc(p.beta[1]);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            Acc d_r = ar * a.w[2 * e] - ai * a.w[2 * e + 1], d_i = ar * a.w[2 * e + 1] + ai * a.w[2 * e];
            if (p.use_c) {
                const Acc cr = c.w[2 * e], ci = p.conjC ? -c.w[2 * e + 1] : c.w[2 * e + 1];
                d_r += br * cr - bi * ci;
                d_i += br * ci + bi * cr;
            }
            d.w[2 * e] = d_r;
            d.w[2 * e + 1] = d_i;
        }
    } else {
        const Acc al = Acc(p.alpha[0]), be = Acc(p.beta[0]);
#pragma unroll
        for (int e = 0; e < V; ++e) {
            Acc v = al * a.w[e];
            if (p.use_c) v += be * c.w[e];
            d.w[e] = v;
        }
    }
    *reinterpret_cast<uint4 *>(static_cast<Acc *>(p.D) + off * W) = d.raw;
}

// Walk the image.  `image` holds BN columns of ImagePitch<BM> elements (W words each); `t` is the
// caller's index among the NT cooperating threads.
template <typename Acc, int W, int BM, int BN, int NT>
__device__ __forceinline__ void store_tile_image(const TiledParams &p, const TileCoords &tc, const Acc *image,
                                                 const int64_t *rowD, const int64_t *colD, int t)
{
    constexpr int P = ImagePitch<BM>::value;
    if (p.split_k > 1) {
        // raw partial sums -> scratch as a dense image [column][row][word] of this CTA's tile
        Acc *ws = static_cast<Acc *>(p.partials) + size_t(blockIdx.x) * (size_t(BM) * BN * W);
#pragma unroll 4
        for (int idx = t; idx < BM * BN * W; idx += NT) {
            const int col = idx / (BM * W), rem = idx % (BM * W);
            ws[idx] = image[col * (P * W) + rem];
        }
        return;
    }
    constexpr int VMAX = 16 / int(sizeof(Acc) * W);      // elements per 16 bytes
    // C may be the same memory as D (in-place update), so the compiler cannot move a load of C
    // above an earlier store to D; the loads of a batch are therefore issued by hand before its
    // stores, which turns a chain of memory round trips into one.
    constexpr int UB = 8;
    if constexpr (VMAX > 1) if (p.vecD >= VMAX && p.vecD % VMAX == 0) {
        constexpr int V = VMAX;
        constexpr int COUNT = (BM / V) * BN;
#pragma unroll 1
        for (int base = t; base < COUNT; base += UB * NT) {
            Pack16<Acc, W, V> c[UB];
            bool ok[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int idx = base + u * NT;
                const int row = (idx % (BM / V)) * V, col = idx / (BM / V);
                ok[u] = idx < COUNT && row < tc.rows_valid && col < tc.cols_valid;   // rows_valid % V == 0 here
                ok[u] = ok[u] && BTC_IN_SPAN(p.spans, 2, rowD[row] + colD[col], V);
                if (ok[u] && p.use_c)
                    c[u].raw = *reinterpret_cast<const uint4 *>(static_cast<const Acc *>(p.C) + (rowD[row] + colD[col]) * W);
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int idx = base + u * NT;
                const int row = (idx % (BM / V)) * V, col = idx / (BM / V);
                if (ok[u]) finish_vector<Acc, W, V>(p, rowD[row] + colD[col], image + size_t(col * P + row) * W, c[u]);
            }
        }
        return;
    }
    {
        constexpr int COUNT = BM * BN;
#pragma unroll 1
        for (int base = t; base < COUNT; base += UB * NT) {
            Acc c_r[UB], c_i[UB];
            bool ok[UB];
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int idx = base + u * NT;
                const int row = idx % BM, col = idx / BM;
                ok[u] = idx < COUNT && row < tc.rows_valid && col < tc.cols_valid;
                ok[u] = ok[u] && BTC_IN_SPAN(p.spans, 2, rowD[row] + colD[col], 1);
                c_r[u] = c_i[u] = Acc(0);
                if (ok[u] && p.use_c) {
                    const Acc *cp = static_cast<const Acc *>(p.C) + (rowD[row] + colD[col]) * W;
                    c_r[u] = cp[0];
                    if (W == 2) c_i[u] = cp[W - 1];
                }
            }
#pragma unroll
            for (int u = 0; u < UB; ++u) {
                const int idx = base + u * NT;
                const int row = idx % BM, col = idx / BM;
                if (ok[u]) {
                    const Acc *w = image + size_t(col * P + row) * W;
                    finish_element<Acc, W>(p, rowD[row] + colD[col], w[0], W == 2 ? w[W - 1] : Acc(0), c_r[u], c_i[u]);
                }
            }
        }
    }
}

// Split-K inside a cluster: every CTA of the cluster has parked the image of its partial tile at the
// same place of its shared memory.  CTA `rank` finishes the rank-th share of the tile's elements: it
// adds the partial values of all CTAs in rank order (so the result does not depend on scheduling; the
// same order as splitk_reduce_kernel) and writes D.  The caller puts a cluster barrier before and after.
template <typename Acc, int W, int BM, int BN, int NT>
__device__ __forceinline__ void splitk_finish_cluster(const TiledParams &p, const TileCoords &tc, const Acc *image,
                                                      const int64_t *rowD, const int64_t *colD, int t)
{
    static_assert(sizeof(Acc) == 8, "distributed shared memory is read in 8-byte words");
    constexpr int P = ImagePitch<BM>::value;
    const int split = p.split_k;
    const int share = (BM * BN + split - 1) / split;
    const int begin = tc.ks * share, end = begin + share < BM * BN ? begin + share : BM * BN;
    const unsigned image0 = static_cast<unsigned>(__cvta_generic_to_shared(image));
    constexpr int UE = 4;
#pragma unroll 1
    for (int base = begin + t; base < end; base += UE * NT) {
        Acc s_r[UE], s_i[UE];
#pragma unroll
        for (int u = 0; u < UE; ++u) s_r[u] = s_i[u] = Acc(0);
        for (int r = 0; r < split; ++r) {
            Acc v_r[UE], v_i[UE];
#pragma unroll
            for (int u = 0; u < UE; ++u) {
                const int idx = base + u * NT;
                const int row = idx % BM, col = idx / BM;
                const unsigned a = cluster_map(image0 + unsigned(col * P + row) * unsigned(W * 8), unsigned(r));
                v_r[u] = idx < end ? cluster_load_f64(a) : Acc(0);
                v_i[u] = (W == 2 && idx < end) ? cluster_load_f64(a + 8u) : Acc(0);
            }
#pragma unroll
            for (int u = 0; u < UE; ++u) { s_r[u] += v_r[u]; s_i[u] += v_i[u]; }
        }
#pragma unroll
        for (int u = 0; u < UE; ++u) {
            const int idx = base + u * NT;
            const int row = idx % BM, col = idx / BM;
            if (idx >= end || row >= tc.rows_valid || col >= tc.cols_valid) continue;
            const int64_t off = rowD[row] + colD[col];
            if (!BTC_IN_SPAN(p.spans, 2, off, 1)) continue;
            Acc c_r = 0, c_i = 0;
            if (p.use_c) {
                const Acc *cp = static_cast<const Acc *>(p.C) + off * W;
                c_r = cp[0];
                if (W == 2) c_i = cp[W - 1];
            }
            finish_element<Acc, W>(p, off, s_r[u], s_i[u], c_r, c_i);
        }
    }
}

// Second pass of split-K for every tiled kernel of one element type: scratch holds, per (batch,
// slice, tile), the dense image [column][row][word] of raw partial sums.  One CTA per (tile,
// batch); slices are added in increasing order, so the result does not depend on scheduling.
template <typename Acc, int W>
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const TiledParams p)
{
    // a wait that gave up in the first pass left slices unwritten: D stays as it was, the error word tells
    if (p.error_word && *static_cast<volatile int32_t *>(p.error_word) != 0) return;
    // blockIdx.x enumerates (chunk of 1024 tile elements, tile, batch), chunk fastest
    const int bm = p.bm, bn = p.bn;
    const int chunks = (bm * bn + 1023) / 1024;
    const int tiles = p.tiles_m * p.tiles_n;
    const int chunk = blockIdx.x % chunks;
    const int tile = (blockIdx.x / chunks) % tiles;
    const int64_t h = blockIdx.x / (chunks * tiles);
    const int tile_m = p.raster_n_fast ? tile / p.tiles_n : tile % p.tiles_m;
    const int tile_n = p.raster_n_fast ? tile % p.tiles_n : tile / p.tiles_m;
    const int64_t m0 = int64_t(tile_m) * bm, n0 = int64_t(tile_n) * bn;
    const int rows_valid = int(imin64(bm, p.M - m0)), cols_valid = int(imin64(bn, p.N - n0));
    const int64_t hD = p.offD_h[h];
    const size_t image = size_t(bm) * bn * W;
    const Acc *ws = static_cast<const Acc *>(p.partials) + (size_t(h) * p.split_k * tiles + tile) * image;
    const size_t slice = size_t(tiles) * image;
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int idx = chunk * 1024 + u * 256 + int(threadIdx.x);
        const int row = idx % bm, col = idx / bm;
        if (idx >= bm * bn || row >= rows_valid || col >= cols_valid) continue;
        const int64_t off = p.offD_m[m0 + row] + hD + p.offD_n[n0 + col];
        if (!BTC_IN_SPAN(p.spans, 2, off, 1)) continue;
        Acc c_r = 0, c_i = 0;
        if (p.use_c) {
            const Acc *cp = static_cast<const Acc *>(p.C) + off * W;
            c_r = cp[0];
            if (W == 2) c_i = cp[W - 1];
        }
        Acc s_r = 0, s_i = 0;
        for (int ks = 0; ks < p.split_k; ++ks) {
            const Acc *src = ws + size_t(ks) * slice + size_t(idx) * W;
            s_r += src[0];
            if (W == 2) s_i += src[W - 1];
        }
        finish_element<Acc, W>(p, off, s_r, s_i, c_r, c_i);
    }
}

}  // namespace btc

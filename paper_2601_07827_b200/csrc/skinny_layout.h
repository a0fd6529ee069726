// Shared-memory layouts of the operand tiles of the short-K streaming kernel (skinny_umma_kernel.cuh),
// usable on the host too: the planner groups the 16-byte pieces of a tile by the 128-byte
// shared-memory line they land in.
#pragma once

#include <cstdint>

#if defined(__CUDACC__)
#define BTC_HD __host__ __device__ __forceinline__
#else
#define BTC_HD inline
#endif

namespace btc {

constexpr int kSkinnyRows = 128;             // rows of an operand tile (BM = BN)
constexpr int kSkinnyBlockBytes = 128 * 128; // one block of 32 k of the N-side tile

// Byte position of a 16-byte piece inside one operand tile of R rows x 32 k in the two layouts the
// tensor core reads (see tiled_umma_tf32x3_kernel.cuh): k-contiguous rows with the 128-byte swizzle
// on 16-byte units; rows-contiguous with the 128-byte swizzle on 32-byte units.
BTC_HD unsigned skinny_piece_kmajor(int row, int k)
{
    return unsigned((row >> 3) * 1024 + (row & 7) * 128 + ((((k >> 2) ^ row) & 7) << 4));
}
BTC_HD unsigned skinny_piece_mnmajor(int row, int k)
{
    const int line = k & 3, unit = ((row & 31) >> 3) ^ line;
    return unsigned(((k >> 2) * (kSkinnyRows / 32) + (row >> 5)) * 512 + line * 128 + unit * 32 + (row & 7) * 4);
}

// Position of 16-byte piece `e` of the M-side tile in its raw shared-memory buffer, and the row and k it
// starts at.  Rows contiguous in memory (dir 0): piece = 4 rows at one k, stored [k][128 rows].
// k contiguous (dir 1): piece = 4 k of one row, stored [row][64 k] with the piece index XORed by
// (row mod 16), so that a quarter-warp reading one piece column of 8 consecutive rows hits 8 banks groups.
BTC_HD unsigned skinny_a_pos(int dir, unsigned e, int &row, int &k)
{
    if (dir == 0) {
        row = int(e & 31u) * 4;
        k = int(e >> 5);
        return unsigned(k * kSkinnyRows + row) * 4u;
    }
    row = int(e & 127u);
    const int k4 = int(e >> 7);
    k = 4 * k4;
    return unsigned(row) * 256u + (unsigned((k4 ^ row) & 15) << 4);
}
// Same for the N-side tile, which sits in the layout the tensor core reads (see piece_kmajor /
// piece_mnmajor): two blocks of 32 k.
BTC_HD unsigned skinny_b_pos(int dir, unsigned e, int &row, int &k)
{
    if (dir == 0) {
        row = int(e & 31u) * 4;
        k = int(e >> 5);
        return unsigned(k >> 5) * unsigned(kSkinnyBlockBytes) + skinny_piece_mnmajor(row, k & 31);
    }
    row = int(e & 127u);
    const int k4 = int(e >> 7);
    k = 4 * k4;
    return unsigned(k4 >> 3) * unsigned(kSkinnyBlockBytes) + skinny_piece_kmajor(row, 4 * (k4 & 7));
}

}  // namespace btc

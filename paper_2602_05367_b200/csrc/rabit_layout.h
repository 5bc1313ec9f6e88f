// Packed device layout of a residual-binary layer (product side; host and device code).
//
// The sign bits of each path are cut into tiles of 32 output rows x 128 input columns.
// One tile is 512 bytes = 32 lanes x 16 bytes, so a warp fetches a tile with one 128-bit
// load per lane, and the four 32-bit words of a lane are exactly the A fragment
// (a0..a3) of an m16n8k32 integer MMA.  Inside every byte the eight bits belong to
// 2 adjacent rows x 4 column sets, so that masking a word with 0x01010101 << p (one
// logic instruction, no shift) yields a valid u8 operand with entries {0, 2^p}:
//
//   lane = 4*gq + tq (gq 0..7, tq 0..3), word a (0..3), byte c (0..3), bit p (0..7)
//     row = 32*rt + 2*(gq + 8*(a & 1)) + (p & 1)
//     col = 128*cg + 32*(p >> 1) + 16*(a >> 1) + 4*tq + c
//
// Tiles are ordered [column slice][row tile][column group inside the slice][path], a slice
// being `slice_cg` consecutive column groups (the last slice may be shorter).  A CTA that
// works on a contiguous range of (slice,row tile) items therefore streams one contiguous
// byte range and needs the activations of one or two slices only.  M is padded to a
// multiple of 32 and N to a multiple of 128 with +1 signs (bit 0) and zero scales.
#ifndef RABIT_LAYOUT_H_
#define RABIT_LAYOUT_H_

#include <stdint.h>
#include <stddef.h>

#if defined(__CUDACC__)
#define RABIT_HD __host__ __device__ __forceinline__
#else
#define RABIT_HD inline
#endif

#define RABIT_MAGIC 0x54494252u /* "RBIT" little endian */
#define RABIT_LAYOUT_VERSION 1
#define RABIT_TILE_ROWS 32
#define RABIT_TILE_COLS 128
#define RABIT_TILE_BYTES 512
#define RABIT_TILE_WORDS 128
#define RABIT_HEADER_BYTES 256
#define RABIT_MAX_K 3
#define RABIT_MAX_GEMV_BATCH 16
#define RABIT_PARTIAL_BATCH 2   /* batch rows the cross-slice partial buffer holds */

struct RabitHeader {            // first 256 bytes of a packed image (little endian)
    uint32_t magic;
    uint32_t version;
    uint32_t K, M, N;
    uint32_t Mp, Np;            // padded extents (multiples of 32 and 128)
    uint32_t n_rt, n_cg;        // row tiles, column groups
    uint32_t slice_cg;          // column groups per slice
    uint32_t n_slices;
    uint32_t reserved0;
    uint64_t off_bits, off_g, off_h, off_partial, off_counters, total_bytes;
    uint8_t pad[RABIT_HEADER_BYTES - 12 * 4 - 6 * 8];
};

struct RabitGeom {              // what kernels need, by value
    int K, M, N, Mp, Np, n_rt, n_cg, slice_cg, n_slices;
};

RABIT_HD size_t rabit_align256(size_t v) { return (v + 255) & ~(size_t)255; }

RABIT_HD int rabit_slice_ncg(const RabitGeom& G, int s) {
    int lo = s * G.slice_cg;
    int hi = lo + G.slice_cg;
    if (hi > G.n_cg) hi = G.n_cg;
    return hi - lo;
}

// Index (in tiles) of tile (slice s, row tile rt, column group q inside the slice, path k).
RABIT_HD size_t rabit_tile_index(const RabitGeom& G, int s, int rt, int q, int k) {
    size_t before = (size_t)G.K * G.n_rt * ((size_t)s * G.slice_cg);
    return before + ((size_t)rt * rabit_slice_ncg(G, s) + q) * G.K + k;
}

#endif  // RABIT_LAYOUT_H_

// Packed device layout of a residual-binary layer, version 2 (product side; host and device code).
//
// The sign bits of each path are cut into tiles of 128 output rows x 32 input columns.
// One tile is 512 bytes = 32 lanes x 16 bytes, so a warp reads a tile with one 128-bit
// access per lane.  The eight bits of every byte belong to eight different 16-row blocks of
// the same input column, so masking a 32-bit word with 0x01010101 << p (one logic
// instruction, no shift) leaves a valid u8 operand word with entries {0, 2^p}, and the
// four masked words of a lane are exactly the A fragment (a0..a3) of an m16n8k32 integer
// MMA over rows 16p .. 16p+15 of the tile:
//
//   lane = 4*gq + tq (gq 0..7, tq 0..3), word a (0..3), byte c (0..3), bit p (0..7)
//     row = 128*rt + 16*p + gq + 8*(a & 1)
//     col = 32*ct + 16*(a >> 1) + 4*tq + c
//
// All eight MMAs of a tile multiply the same 32 columns, so they share one B fragment.
// Tiles are stored in the linear order  pos = (rt * K + k) * n_ct + ct  (row tile, path,
// column tile): the K paths of a row tile are interleaved strip by strip, and any contiguous
// range of positions is one contiguous byte range, which is what a CTA streams.
// M is padded to a multiple of 128 with +1 signs (bit 0) and zero scales; N must be a
// multiple of 32 and is not padded.
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
#define RABIT_LAYOUT_VERSION 2
#define RABIT_TILE_ROWS 128
#define RABIT_TILE_COLS 32
#define RABIT_TILE_BYTES 512
#define RABIT_HEADER_BYTES 256
#define RABIT_MAX_K 3
#define RABIT_MAX_GEMV_BATCH 16
#define RABIT_PARTIAL_BATCH 4   /* batch rows the cross-CTA partial buffer holds */
#define RABIT_MAX_GRID 320      /* most CTAs a GEMV launch may use (sizes the partial buffer) */

struct RabitHeader {            // first 256 bytes of a packed image (little endian)
    uint32_t magic;
    uint32_t version;
    uint32_t K, M, N;
    uint32_t Mp;                // M rounded up to a multiple of 128
    uint32_t n_rt, n_ct;        // row tiles (Mp/128), column tiles (N/32)
    uint32_t max_grid;          // RABIT_MAX_GRID at pack time
    uint32_t partial_batch;     // RABIT_PARTIAL_BATCH at pack time
    uint32_t hmax_bits[4];      // fp32 bit pattern of max_j |h_k[j]| per path (0 for unused paths)
    uint32_t reserved[2];
    uint64_t off_bits, off_g, off_h, off_partial, off_flags, total_bytes;
    uint8_t pad[RABIT_HEADER_BYTES - 16 * 4 - 6 * 8];
};

struct RabitGeom {              // what kernels need, by value
    int K, M, N, Mp, n_rt, n_ct;
    float hmax[RABIT_MAX_K];
};

RABIT_HD size_t rabit_align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Linear position of tile (row tile rt, path k, column tile ct).
RABIT_HD size_t rabit_tile_pos(const RabitGeom& G, int rt, int k, int ct) {
    return ((size_t)rt * G.K + k) * G.n_ct + ct;
}

#endif  // RABIT_LAYOUT_H_

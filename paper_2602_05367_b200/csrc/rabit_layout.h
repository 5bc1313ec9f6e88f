// Packed device layout of a residual-binary layer, version 3 (product side; host and device code).
//
// The image carries the sign bits in two arrangements, one per kernel family, plus the scales and
// the scratch the decode kernels need:
//
//   header | sign tiles | g fp16 [K][Mp] | h fp16 [K][N] | fp32 partial scratch | flags + status |
//   look-up blocks | u64 accumulate words
//
// (1) Sign tiles (tensor-core kernels: the f16 and integer-MMA GEMVs of batches 3..16 and the tcgen05 GEMM).
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
//
// (2) Look-up blocks (the table-driven decode GEMV of batches 1..2).  Here a byte holds the signs of
// eight consecutive input columns of ONE row (bit b <-> column 8*group + b), so a byte is the index
// of a 256-entry table of partial sums over those eight columns.  The input dimension is cut into
// slices of 256 columns (32 byte groups), the output dimension into row blocks of 32 rows (one row
// per lane).  A block (slice cs, row block rb) holds K consecutive 1 KB parts, one per path; a part
// is 2 halves x 32 lanes x 16 bytes, and byte q of (half hf, lane l) is the byte group
//
//     group = (16*hf + q + l) mod 32        row = 32*rb + l        columns 256*cs + 8*group .. +7
//
// i.e. every lane walks the 32 groups of its row in an order rotated by its lane index, so that the
// 32 table look-ups of a warp step fall into 32 different shared-memory banks.  Blocks are stored in
// the order  pos = cs * n_rb + rb  (slice-major), K KB each: a contiguous range of positions is a
// contiguous byte range and keeps one table in use for as long as possible.  Columns beyond N
// (when N is not a multiple of 256) and rows beyond M hold bit 0.
//
// M is padded to a multiple of 128 with +1 signs (bit 0) and zero scales; N must be a
// multiple of 32.  The accumulate words (u64 [RABIT_LUT_MAX_BATCH][Mp]) rest at zero.
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
#define RABIT_LAYOUT_VERSION 3
#define RABIT_TILE_ROWS 128
#define RABIT_TILE_COLS 32
#define RABIT_TILE_BYTES 512
#define RABIT_HEADER_BYTES 256
#define RABIT_MAX_K 3
#define RABIT_MAX_GEMV_BATCH 16
#define RABIT_PARTIAL_BATCH 4   /* batch rows the cross-CTA partial buffer holds */
#define RABIT_MAX_GRID 320      /* most CTAs a GEMV launch may use (sizes the partial buffer) */
#define RABIT_LUT_ROWS 32       /* output rows of a look-up block (one per lane) */
#define RABIT_LUT_COLS 256      /* input columns of a slice (32 byte groups) */
#define RABIT_LUT_PART_BYTES 1024   /* one path of one block */
#define RABIT_LUT_MAX_BATCH 16  /* batch rows the accumulate words provide for */
#define RABIT_LUT_MAX_SLICES 255    /* the arrival count of an accumulate word has eight bits */

struct RabitHeader {            // first 256 bytes of a packed image (little endian)
    uint32_t magic;
    uint32_t version;
    uint32_t K, M, N;
    uint32_t Mp;                // M rounded up to a multiple of 128
    uint32_t n_rt, n_ct;        // row tiles (Mp/128), column tiles (N/32)
    uint32_t max_grid;          // RABIT_MAX_GRID at pack time
    uint32_t partial_batch;     // RABIT_PARTIAL_BATCH at pack time
    uint32_t hmax_bits[4];      // fp32 bit pattern of max_j |h_k[j]| per path (0 for unused paths)
    uint32_t n_rb, n_cs;        // look-up row blocks (Mp/32) and column slices (ceil(N/256))
    uint32_t fix_bits;          // magnitude bits of one fixed-point contribution to an accumulate word
    int32_t unit_exp;           // one fixed-point unit is 2^unit_exp
    uint32_t reserved[2];
    uint64_t off_bits, off_g, off_h, off_partial, off_flags, off_lut, off_acc, total_bytes;
    uint8_t pad[RABIT_HEADER_BYTES - 20 * 4 - 8 * 8];
};

struct RabitGeom {              // what kernels need, by value
    int K, M, N, Mp, n_rt, n_ct;
    float hmax[RABIT_MAX_K];
    int n_rb, n_cs;
    int fix_bits, unit_exp;
};

RABIT_HD size_t rabit_align256(size_t v) { return (v + 255) & ~(size_t)255; }

// Linear position of tile (row tile rt, path k, column tile ct).
RABIT_HD size_t rabit_tile_pos(const RabitGeom& G, int rt, int k, int ct) {
    return ((size_t)rt * G.K + k) * G.n_ct + ct;
}

// Byte offset, inside the look-up section, of the byte that holds columns 8*cb .. 8*cb+7 of `row` in path k.
RABIT_HD size_t rabit_lut_byte_offset(const RabitGeom& G, int k, int row, int cb) {
    const int cs = cb >> 5, group = cb & 31, rb = row >> 5, l = row & 31;
    const int s = (group - l) & 31;
    return (((size_t)cs * G.n_rb + rb) * G.K + k) * RABIT_LUT_PART_BYTES + (size_t)(s >> 4) * 512 + l * 16 + (s & 15);
}

#endif  // RABIT_LAYOUT_H_

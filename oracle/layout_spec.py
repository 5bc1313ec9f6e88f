"""Reference statement of the packed device layout (version 3).  TEST INFRASTRUCTURE ONLY.

Written from the layout's definition, independently of the library's packer, so that the
library image can be compared byte for byte.  The paper fixes only the sign -> bit rule
(Appendix "Weight Packing": +1 -> 0, -1 -> 1); the arrangement below is this build's.

Image = header (256 B) | sign tiles | g fp16 [K][Mp] | h fp16 [K][N] | fp32 partial scratch
[n_rt*K + max_grid][partial_batch][128] | u32 flags [n_rt*K + max_grid] + one status word |
look-up blocks | u64 accumulate words [16][Mp]; every section starts on a 256-byte boundary;
padding, flags (reserved), status and accumulate words are zero, the partial scratch section is
filled with 0xFF bytes (its resting state: "nothing written yet").
Mp = M rounded up to 128; padded signs are +1 (bit 0), padded scales 0; N is a multiple of
32 and is not padded in the tile section.  The header also records max_j |h_k[j]| per path as an
fp32 bit pattern (the integer kernels derive their fixed-point scale from it) and the fixed-point
grid of the accumulate words (see ``fixed_point_grid``).

The signs are stored twice, once per kernel family.

A tile holds 128 rows x 32 columns of one path in 512 bytes.  Byte ``16*lane + 4*a + c`` of
a tile (lane = 4*gq + tq) has, in bit p,

    row = 128*rt + 16*p + gq + 8*(a & 1)
    col = 32*ct + 16*(a >> 1) + 4*tq + c

Tiles are stored at position ``(rt*K + k)*n_ct + ct`` (row tile, path, column tile).

Look-up blocks: the input columns are cut into slices of 256 (``n_cs = ceil(N/256)``; columns
beyond N hold bit 0), the padded rows into blocks of 32 (``n_rb = Mp/32``).  A byte holds eight
consecutive columns of one row, bit b <-> column ``8*group + b`` of the slice.  Block (cs, rb)
sits at position ``cs*n_rb + rb`` and holds K parts of 1024 bytes (path 0, 1, ...); inside a part,
byte ``512*hf + 16*l + q`` (hf 0..1, l 0..31, q 0..15) is

    row = 32*rb + l,   group = (16*hf + q + l) mod 32      (columns 256*cs + 8*group .. +7)
"""
from __future__ import annotations

import struct

import numpy as np

MAGIC = 0x54494252
VERSION = 3
HEADER_BYTES = 256
TILE_BYTES = 512
TILE_ROWS = 128
TILE_COLS = 32
MAX_GRID = 320
PARTIAL_BATCH = 4
LUT_ROWS = 32
LUT_COLS = 256
LUT_PART_BYTES = 1024
LUT_MAX_BATCH = 16
_HEADER_FMT = "<14I2IIi2I8Q"
_HEADER_KEYS = ["magic", "version", "K", "M", "N", "Mp", "n_rt", "n_ct", "max_grid", "partial_batch",
                "hmax0", "hmax1", "hmax2", "hmax3", "n_rb", "n_cs", "fix_bits", "unit_exp", "reserved0", "reserved1",
                "off_bits", "off_g", "off_h", "off_partial", "off_flags", "off_lut", "off_acc", "total_bytes"]


def _align256(v: int) -> int:
    return (v + 255) // 256 * 256


def geometry(K: int, M: int, N: int) -> dict:
    Mp = (M + TILE_ROWS - 1) // TILE_ROWS * TILE_ROWS
    n_rt, n_ct = Mp // TILE_ROWS, N // TILE_COLS
    n_rb, n_cs = Mp // LUT_ROWS, (N + LUT_COLS - 1) // LUT_COLS
    geo = dict(K=K, M=M, N=N, Mp=Mp, n_rt=n_rt, n_ct=n_ct, n_rb=n_rb, n_cs=n_cs)
    off = HEADER_BYTES
    geo["off_bits"] = off; off = _align256(off + K * n_rt * n_ct * TILE_BYTES)
    geo["off_g"] = off; off = _align256(off + K * Mp * 2)
    geo["off_h"] = off; off = _align256(off + K * N * 2)
    geo["off_partial"] = off; off = _align256(off + (n_rt * K + MAX_GRID) * PARTIAL_BATCH * TILE_ROWS * 4)
    geo["off_flags"] = off; off = _align256(off + (n_rt * K + MAX_GRID) * 4 + 4)
    geo["off_lut"] = off; off = _align256(off + n_cs * n_rb * K * LUT_PART_BYTES)
    geo["off_acc"] = off; off = _align256(off + LUT_MAX_BATCH * Mp * 8)
    geo["total_bytes"] = off
    return geo


def fixed_point_grid(g16: np.ndarray, h16: np.ndarray, n_cs: int):
    """(fix_bits, unit_exp) of the accumulate words.

    The table-driven kernel adds one partial sum per 256-column slice to a 64-bit word per output row
    with an integer atomic.  For any finite fp16 activation, |partial sum| <= bound with
    ``bound = 65504 * max_i sum_k |g_k[i]| * max_{k, slice} sum_{j in slice} |h_k[j]|``.
    fix_bits = 54 - ceil(log2(n_cs)) magnitude bits per contribution (the biased contributions of all
    slices then stay below 2^55); the grid covers 2^e with bound < 2^(e-1) (one spare bit), e clipped to
    [-40, 100]; unit_exp = e - fix_bits.  A zero or non-finite bound gives e = 0.
    """
    g = np.abs(g16.astype(np.float64))
    h = np.abs(h16.astype(np.float64))
    gsum = g.sum(axis=0).max()
    N = h.shape[1]
    hsum = max(h[k, j0:j0 + LUT_COLS].sum() for k in range(h.shape[0]) for j0 in range(0, N, LUT_COLS))
    clog = 0
    while (1 << clog) < n_cs:
        clog += 1
    fix_bits = 54 - clog
    bound = 65504.0 * gsum * hsum
    e = 0
    if np.isfinite(bound) and bound > 0.0:
        _, ex = np.frexp(bound)          # bound = m * 2^ex, 0.5 <= m < 1
        e = int(ex) + 1
    e = max(-40, min(100, e))
    return fix_bits, e - fix_bits


def header_bytes(geo: dict, hmax_bits, fix_bits: int, unit_exp: int) -> bytes:
    hm = list(hmax_bits) + [0] * (4 - len(hmax_bits))
    head = struct.pack(_HEADER_FMT, MAGIC, VERSION, geo["K"], geo["M"], geo["N"], geo["Mp"], geo["n_rt"], geo["n_ct"],
                       MAX_GRID, PARTIAL_BATCH, hm[0], hm[1], hm[2], hm[3], geo["n_rb"], geo["n_cs"], fix_bits, unit_exp, 0, 0,
                       geo["off_bits"], geo["off_g"], geo["off_h"], geo["off_partial"], geo["off_flags"],
                       geo["off_lut"], geo["off_acc"], geo["total_bytes"])
    return head + bytes(HEADER_BYTES - len(head))


def _lut_of_plane(plane: np.ndarray, M: int, N: int, Mp: int) -> np.ndarray:
    """uint8 [n_cs][n_rb][1024] for one path, straight from the definition of a part."""
    n_rb, n_cs = Mp // LUT_ROWS, (N + LUT_COLS - 1) // LUT_COLS
    bits = np.unpackbits(plane.astype("<u4").view(np.uint8), axis=-1, bitorder="little")[:, :N]   # [M][N] 0/1
    full = np.zeros((Mp, n_cs * LUT_COLS), dtype=np.uint8)
    full[:M, :N] = bits
    groups = np.packbits(full.reshape(Mp, n_cs * 32, 8), axis=-1, bitorder="little")[..., 0]       # [Mp][n_cs*32] bytes
    out = np.zeros((n_cs, n_rb, LUT_PART_BYTES), dtype=np.uint8)
    by_block = groups.reshape(n_rb, 32, n_cs, 32)                        # [rb][l][cs][group]
    for hf in range(2):
        for l in range(32):
            for q in range(16):
                group = (16 * hf + q + l) % 32
                out[:, :, 512 * hf + 16 * l + q] = by_block[:, l, :, group].T     # [cs][rb]
    return out


def read_header(image: np.ndarray) -> dict:
    vals = struct.unpack(_HEADER_FMT, bytes(image[:struct.calcsize(_HEADER_FMT)]))
    return dict(zip(_HEADER_KEYS, vals))


def _tiles_of_plane(plane: np.ndarray, M: int, N: int, Mp: int) -> np.ndarray:
    """uint8 [n_rt][n_ct][512] for one path."""
    bits = np.unpackbits(plane.astype("<u4").view(np.uint8), axis=-1, bitorder="little")[:, :N]   # [M][N] 0/1
    full = np.zeros((Mp, N), dtype=np.uint8)
    full[:M] = bits
    n_rt, n_ct = Mp // TILE_ROWS, N // TILE_COLS
    # row = 128*rt + 16*p + 8*alo + gq           -> axes (rt, p, alo, gq)
    # col = 32*ct + 16*ah + 4*tq + c             -> axes (ct, ah, tq, c)
    v = full.reshape(n_rt, 8, 2, 8, n_ct, 2, 4, 4)
    #                 0   1  2  3   4    5  6  7
    #                 rt  p alo gq  ct   ah tq c
    v = v.transpose(0, 4, 3, 6, 5, 2, 7, 1)          # rt ct gq tq ah alo c p
    by = np.packbits(v, axis=-1, bitorder="little")[..., 0]   # bit p of the byte <- axis p
    return by.reshape(n_rt, n_ct, TILE_BYTES)        # offset = 64*gq + 16*tq + 8*ah + 4*alo + c = 16*lane + 4*a + c


def pack_spec(planes: np.ndarray, g: np.ndarray, h: np.ndarray) -> np.ndarray:
    planes = np.asarray(planes, dtype=np.uint32)
    K, M, W = planes.shape
    N = W * 32
    geo = geometry(K, M, N)
    h16 = np.asarray(h, dtype=np.float16)
    g16 = np.asarray(g, dtype=np.float16)
    hmax_bits = [int(np.abs(h16[k].astype(np.float32)).max().view(np.uint32)) for k in range(K)]
    img = np.zeros(geo["total_bytes"], dtype=np.uint8)
    fix_bits, unit_exp = fixed_point_grid(g16, h16, geo["n_cs"])
    img[:HEADER_BYTES] = np.frombuffer(header_bytes(geo, hmax_bits, fix_bits, unit_exp), dtype=np.uint8)
    lut = np.stack([_lut_of_plane(planes[k], M, N, geo["Mp"]) for k in range(K)], axis=2)   # [cs][rb][k][1024]
    img[geo["off_lut"]:geo["off_lut"] + lut.size] = lut.reshape(-1)
    tiles = np.stack([_tiles_of_plane(planes[k], M, N, geo["Mp"]) for k in range(K)], axis=1)   # [rt][k][ct][512]
    flat = tiles.reshape(-1)
    img[geo["off_bits"]:geo["off_bits"] + flat.size] = flat
    img[geo["off_partial"]:geo["off_flags"]] = 0xFF
    gp = np.zeros((K, geo["Mp"]), dtype=np.uint16); gp[:, :M] = g16.view(np.uint16)
    img[geo["off_g"]:geo["off_g"] + gp.nbytes] = gp.view(np.uint8).reshape(-1)
    hp = np.ascontiguousarray(h16.view(np.uint16))
    img[geo["off_h"]:geo["off_h"] + hp.nbytes] = hp.view(np.uint8).reshape(-1)
    return img


def unpack_lut_spec(img: np.ndarray) -> np.ndarray:
    """Planes recovered from the look-up blocks alone, byte by byte from the definition (slow)."""
    hd = read_header(img)
    K, M, N, n_rb, n_cs = hd["K"], hd["M"], hd["N"], hd["n_rb"], hd["n_cs"]
    planes = np.zeros((K, M, N // 32), dtype=np.uint32)
    sec = img[hd["off_lut"]:hd["off_lut"] + n_cs * n_rb * K * LUT_PART_BYTES].reshape(n_cs, n_rb, K, LUT_PART_BYTES)
    for cs, rb, k, off in zip(*np.nonzero(sec)):
        byte = int(sec[cs, rb, k, off])
        hf, l, q = off // 512, (off % 512) // 16, off % 16
        row, group = 32 * rb + l, (16 * hf + q + l) % 32
        for b in range(8):
            if (byte >> b) & 1:
                col = 256 * cs + 8 * group + b
                assert row < M and col < N, "padding bit set"
                planes[k, row, col // 32] |= np.uint32(1 << (col % 32))
    return planes


def unpack_spec(img: np.ndarray):
    """Inverse of pack_spec, bit by bit from the definition (slow; small shapes only)."""
    hd = read_header(img)
    K, M, N, n_rt, n_ct = hd["K"], hd["M"], hd["N"], hd["n_rt"], hd["n_ct"]
    planes = np.zeros((K, M, N // 32), dtype=np.uint32)
    for rt in range(n_rt):
        for k in range(K):
            for ct in range(n_ct):
                pos = (rt * K + k) * n_ct + ct
                tile = img[hd["off_bits"] + pos * TILE_BYTES: hd["off_bits"] + (pos + 1) * TILE_BYTES]
                for off in np.flatnonzero(tile):
                    byte = int(tile[off])
                    lane, a, c = off // 16, (off % 16) // 4, off % 4
                    gq, tq = lane // 4, lane % 4
                    for p in range(8):
                        if (byte >> p) & 1:
                            row = 128 * rt + 16 * p + gq + 8 * (a & 1)
                            col = 32 * ct + 16 * (a >> 1) + 4 * tq + c
                            assert row < M and col < N, "padding bit set"
                            planes[k, row, col // 32] |= np.uint32(1 << (col % 32))
    g = img[hd["off_g"]:hd["off_g"] + K * hd["Mp"] * 2].view(np.uint16).reshape(K, hd["Mp"])[:, :M]
    h = img[hd["off_h"]:hd["off_h"] + K * N * 2].view(np.uint16).reshape(K, N)
    return planes, g.view(np.float16).copy(), h.view(np.float16).copy()

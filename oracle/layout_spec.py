"""Reference statement of the packed device layout (version 2).  TEST INFRASTRUCTURE ONLY.

Written from the layout's definition, independently of the library's packer, so that the
library image can be compared byte for byte.  The paper fixes only the sign -> bit rule
(Appendix "Weight Packing": +1 -> 0, -1 -> 1); the arrangement below is this build's.

Image = header (256 B) | sign tiles | g fp16 [K][Mp] | h fp16 [K][N] | fp32 partial scratch
[n_rt*K + max_grid][partial_batch][128] | u32 flags [n_rt*K + max_grid] + one status word; every
section starts on a 256-byte boundary; padding, flags (reserved) and status are zero, the partial
scratch section is filled with 0xFF bytes (its resting state: "nothing written yet").
Mp = M rounded up to 128; padded signs are +1 (bit 0), padded scales 0; N is a multiple of
32 and is not padded.  The header also records max_j |h_k[j]| per path as an fp32 bit
pattern (the kernels derive their fixed-point scale from it).

A tile holds 128 rows x 32 columns of one path in 512 bytes.  Byte ``16*lane + 4*a + c`` of
a tile (lane = 4*gq + tq) has, in bit p,

    row = 128*rt + 16*p + gq + 8*(a & 1)
    col = 32*ct + 16*(a >> 1) + 4*tq + c

Tiles are stored at position ``(rt*K + k)*n_ct + ct`` (row tile, path, column tile).
"""
from __future__ import annotations

import struct

import numpy as np

MAGIC = 0x54494252
VERSION = 2
HEADER_BYTES = 256
TILE_BYTES = 512
TILE_ROWS = 128
TILE_COLS = 32
MAX_GRID = 320
PARTIAL_BATCH = 4
_HEADER_FMT = "<16I6Q"
_HEADER_KEYS = ["magic", "version", "K", "M", "N", "Mp", "n_rt", "n_ct", "max_grid", "partial_batch",
                "hmax0", "hmax1", "hmax2", "hmax3", "reserved0", "reserved1",
                "off_bits", "off_g", "off_h", "off_partial", "off_flags", "total_bytes"]


def _align256(v: int) -> int:
    return (v + 255) // 256 * 256


def geometry(K: int, M: int, N: int) -> dict:
    Mp = (M + TILE_ROWS - 1) // TILE_ROWS * TILE_ROWS
    n_rt, n_ct = Mp // TILE_ROWS, N // TILE_COLS
    geo = dict(K=K, M=M, N=N, Mp=Mp, n_rt=n_rt, n_ct=n_ct)
    off = HEADER_BYTES
    geo["off_bits"] = off; off = _align256(off + K * n_rt * n_ct * TILE_BYTES)
    geo["off_g"] = off; off = _align256(off + K * Mp * 2)
    geo["off_h"] = off; off = _align256(off + K * N * 2)
    geo["off_partial"] = off; off = _align256(off + (n_rt * K + MAX_GRID) * PARTIAL_BATCH * TILE_ROWS * 4)
    geo["off_flags"] = off; off = _align256(off + (n_rt * K + MAX_GRID) * 4 + 4)
    geo["total_bytes"] = off
    return geo


def header_bytes(geo: dict, hmax_bits) -> bytes:
    hm = list(hmax_bits) + [0] * (4 - len(hmax_bits))
    head = struct.pack(_HEADER_FMT, MAGIC, VERSION, geo["K"], geo["M"], geo["N"], geo["Mp"], geo["n_rt"], geo["n_ct"],
                       MAX_GRID, PARTIAL_BATCH, hm[0], hm[1], hm[2], hm[3], 0, 0,
                       geo["off_bits"], geo["off_g"], geo["off_h"], geo["off_partial"], geo["off_flags"],
                       geo["total_bytes"])
    return head + bytes(HEADER_BYTES - len(head))


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
    img[:HEADER_BYTES] = np.frombuffer(header_bytes(geo, hmax_bits), dtype=np.uint8)
    tiles = np.stack([_tiles_of_plane(planes[k], M, N, geo["Mp"]) for k in range(K)], axis=1)   # [rt][k][ct][512]
    flat = tiles.reshape(-1)
    img[geo["off_bits"]:geo["off_bits"] + flat.size] = flat
    img[geo["off_partial"]:geo["off_flags"]] = 0xFF
    gp = np.zeros((K, geo["Mp"]), dtype=np.uint16); gp[:, :M] = g16.view(np.uint16)
    img[geo["off_g"]:geo["off_g"] + gp.nbytes] = gp.view(np.uint8).reshape(-1)
    hp = np.ascontiguousarray(h16.view(np.uint16))
    img[geo["off_h"]:geo["off_h"] + hp.nbytes] = hp.view(np.uint8).reshape(-1)
    return img


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

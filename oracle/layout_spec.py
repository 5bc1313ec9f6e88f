"""Reference statement of the packed device layout (version 1).  TEST INFRASTRUCTURE ONLY.

Written from the layout's definition, independently of the library's packer, so that the
library image can be compared byte for byte.  The paper fixes only the sign -> bit rule
(Appendix "Weight Packing": +1 -> 0, -1 -> 1); the arrangement below is this build's.

Image = header (256 B) | sign tiles | g fp16 [K][Mp] | h fp16 [K][Np] | fp32 scratch
[2][n_slices][Mp] | u32 counters [n_rt]; every section starts on a 256-byte boundary; padding,
scratch and counters are zero.  Mp = M rounded up to 32, Np = N rounded up to 128; padded
signs are +1 (bit 0), padded scales 0.

A tile holds 32 rows x 128 columns of one path in 512 bytes.  Byte ``16*lane + 4*a + c`` of
a tile (lane = 4*gq + tq) has, in bit p,

    row = 32*rt + 2*(gq + 8*(a & 1)) + (p & 1)
    col = 128*cg + 32*(p >> 1) + 16*(a >> 1) + 4*tq + c

Tiles are stored in the order [slice][row tile][column group inside slice][path]; a slice
is ``slice_cg`` consecutive column groups (the last one may be shorter).  ``slice_cg`` is a
free parameter of the format, recorded in the header.
"""
from __future__ import annotations

import struct

import numpy as np

MAGIC = 0x54494252
VERSION = 1
HEADER_BYTES = 256
TILE_BYTES = 512


def _align256(v: int) -> int:
    return (v + 255) // 256 * 256


def geometry(K: int, M: int, N: int, slice_cg: int) -> dict:
    Mp = (M + 31) // 32 * 32
    Np = (N + 127) // 128 * 128
    n_rt, n_cg = Mp // 32, Np // 128
    n_slices = (n_cg + slice_cg - 1) // slice_cg
    off = HEADER_BYTES
    geo = dict(K=K, M=M, N=N, Mp=Mp, Np=Np, n_rt=n_rt, n_cg=n_cg, slice_cg=slice_cg, n_slices=n_slices)
    geo["off_bits"] = off; off = _align256(off + K * n_rt * n_cg * TILE_BYTES)
    geo["off_g"] = off; off = _align256(off + K * Mp * 2)
    geo["off_h"] = off; off = _align256(off + K * Np * 2)
    geo["off_partial"] = off; off = _align256(off + 2 * n_slices * Mp * 4)
    geo["off_counters"] = off; off = _align256(off + n_rt * 4)
    geo["total_bytes"] = off
    return geo


def header_bytes(geo: dict) -> bytes:
    head = struct.pack("<12I6Q", MAGIC, VERSION, geo["K"], geo["M"], geo["N"], geo["Mp"], geo["Np"],
                       geo["n_rt"], geo["n_cg"], geo["slice_cg"], geo["n_slices"], 0,
                       geo["off_bits"], geo["off_g"], geo["off_h"], geo["off_partial"], geo["off_counters"],
                       geo["total_bytes"])
    return head + bytes(HEADER_BYTES - len(head))


def read_header(image: np.ndarray) -> dict:
    vals = struct.unpack("<12I6Q", bytes(image[:96]))
    keys = ["magic", "version", "K", "M", "N", "Mp", "Np", "n_rt", "n_cg", "slice_cg", "n_slices", "reserved0",
            "off_bits", "off_g", "off_h", "off_partial", "off_counters", "total_bytes"]
    return dict(zip(keys, vals))


def _tiles_of_plane(plane: np.ndarray, M: int, N: int, Mp: int, Np: int) -> np.ndarray:
    """uint8 [n_rt][n_cg][512] for one path."""
    bits = np.unpackbits(plane.astype("<u4").view(np.uint8), axis=-1, bitorder="little")[:, :N]   # [M][N] 0/1
    full = np.zeros((Mp, Np), dtype=np.uint8)
    full[:M, :N] = bits
    n_rt, n_cg = Mp // 32, Np // 128
    # row  = 32*rt + 16*alo + 2*gq + rg          -> axes (rt, alo, gq, rg)
    # col  = 128*cg + 32*cs + 16*ah + 4*tq + c   -> axes (cg, cs, ah, tq, c)
    v = full.reshape(n_rt, 2, 8, 2, n_cg, 4, 2, 4, 4)
    #                 0   1  2  3   4   5  6  7  8
    #                 rt alo gq rg  cg  cs ah tq c
    v = v.transpose(0, 4, 2, 7, 6, 1, 8, 5, 3)       # rt cg gq tq ah alo c cs rg
    v = v.reshape(n_rt, n_cg, 8, 4, 2, 2, 4, 8)      # last axis: p = 2*cs + rg
    by = np.packbits(v, axis=-1, bitorder="little")[..., 0]   # rt cg gq tq ah alo c
    return by.reshape(n_rt, n_cg, TILE_BYTES)        # offset = 64*gq + 16*tq + 8*ah + 4*alo + c = 16*lane + 4*a + c


def pack_spec(planes: np.ndarray, g: np.ndarray, h: np.ndarray, slice_cg: int) -> np.ndarray:
    planes = np.asarray(planes, dtype=np.uint32)
    K, M, W = planes.shape
    N = W * 32
    geo = geometry(K, M, N, slice_cg)
    img = np.zeros(geo["total_bytes"], dtype=np.uint8)
    img[:HEADER_BYTES] = np.frombuffer(header_bytes(geo), dtype=np.uint8)
    tiles = [_tiles_of_plane(planes[k], M, N, geo["Mp"], geo["Np"]) for k in range(K)]
    pos = geo["off_bits"]
    n_rt, n_cg = geo["n_rt"], geo["n_cg"]
    for s in range(geo["n_slices"]):
        lo, hi = s * slice_cg, min(n_cg, (s + 1) * slice_cg)
        block = np.stack([tiles[k][:, lo:hi, :] for k in range(K)], axis=2)    # [rt][q][k][512]
        flat = block.reshape(-1)
        img[pos:pos + flat.size] = flat
        pos += flat.size
    g16 = np.zeros((K, geo["Mp"]), dtype=np.uint16); g16[:, :M] = np.asarray(g, dtype=np.float16).view(np.uint16)
    h16 = np.zeros((K, geo["Np"]), dtype=np.uint16); h16[:, :N] = np.asarray(h, dtype=np.float16).view(np.uint16)
    img[geo["off_g"]:geo["off_g"] + g16.nbytes] = g16.view(np.uint8).reshape(-1)
    img[geo["off_h"]:geo["off_h"] + h16.nbytes] = h16.view(np.uint8).reshape(-1)
    return img


def unpack_spec(img: np.ndarray):
    """Inverse of pack_spec, bit by bit from the definition (slow; small shapes only)."""
    hd = read_header(img)
    K, M, N, n_rt, n_cg, slice_cg = hd["K"], hd["M"], hd["N"], hd["n_rt"], hd["n_cg"], hd["slice_cg"]
    planes = np.zeros((K, M, N // 32), dtype=np.uint32)
    for s in range(hd["n_slices"]):
        lo, hi = s * slice_cg, min(n_cg, (s + 1) * slice_cg)
        ncg = hi - lo
        for rt in range(n_rt):
            for q in range(ncg):
                for k in range(K):
                    ti = K * n_rt * s * slice_cg + (rt * ncg + q) * K + k
                    tile = img[hd["off_bits"] + ti * TILE_BYTES: hd["off_bits"] + (ti + 1) * TILE_BYTES]
                    for off in range(TILE_BYTES):
                        byte = int(tile[off])
                        if not byte:
                            continue
                        lane, a, c = off // 16, (off % 16) // 4, off % 4
                        gq, tq = lane // 4, lane % 4
                        for p in range(8):
                            if (byte >> p) & 1:
                                row = 32 * rt + 2 * (gq + 8 * (a & 1)) + (p & 1)
                                col = 128 * (lo + q) + 32 * (p >> 1) + 16 * (a >> 1) + 4 * tq + c
                                assert row < M and col < N, "padding bit set"
                                planes[k, row, col // 32] |= np.uint32(1 << (col % 32))
    g = img[hd["off_g"]:hd["off_g"] + K * hd["Mp"] * 2].view(np.uint16).reshape(K, hd["Mp"])[:, :M]
    h = img[hd["off_h"]:hd["off_h"] + K * hd["Np"] * 2].view(np.uint16).reshape(K, hd["Np"])[:, :N]
    return planes, g.view(np.float16).copy(), h.view(np.float16).copy()

"""CPU-side tests of the product's host logic: the packed layout (bit-exact against the
reference statement of the format), its round trip, argument checking, and that the C-ABI
library exports every symbol the header declares.  No GPU is touched."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2602_05367_b200 as rabit
from paper_2602_05367_b200 import binding
from oracle import layout_spec as spec
from synth import make_layer, make_planes_constant

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

SHAPES = [(1, 32, 32), (2, 32, 128), (2, 64, 256), (2, 100, 160), (3, 33, 1056), (2, 160, 640), (1, 7, 96),
          (2, 256, 1184)]


@pytest.mark.parametrize("K,M,N", SHAPES)
def test_library_image_equals_spec(K, M, N):
    L = make_layer(M, N, K, key=(80, K, M, N))
    img = rabit.pack_host(L.planes, L.g, L.h)
    hd = spec.read_header(img)
    assert hd["magic"] == spec.MAGIC and hd["version"] == rabit.layout_version() == spec.VERSION
    want = spec.pack_spec(L.planes, L.g, L.h)
    assert img.nbytes == want.nbytes == rabit.packed_bytes(K, M, N)
    assert np.array_equal(img, want)


@pytest.mark.parametrize("K,M,N", SHAPES)
def test_round_trip_bit_exact(K, M, N):
    L = make_layer(M, N, K, key=(81, K, M, N))
    img = rabit.pack_host(L.planes, L.g, L.h)
    planes, g, h = rabit.unpack_host(img, K, M, N)
    assert np.array_equal(planes, L.planes)
    assert np.array_equal(g.view(np.uint16), L.g.view(np.uint16))
    assert np.array_equal(h.view(np.uint16), L.h.view(np.uint16))
    # the reference unpacker reads the library image the same way
    if M * N <= 64 * 256:
        p2, g2, h2 = spec.unpack_spec(img)
        assert np.array_equal(p2, L.planes) and np.array_equal(g2.view(np.uint16), L.g.view(np.uint16))
        assert np.array_equal(h2.view(np.uint16), L.h.view(np.uint16))


def test_spec_round_trip_and_library_reads_spec_image():
    L = make_layer(70, 640, 2, key=(82,))
    img = spec.pack_spec(L.planes, L.g, L.h)
    planes, g, h = spec.unpack_spec(img)
    assert np.array_equal(planes, L.planes)
    assert np.array_equal(g.view(np.uint16), L.g.view(np.uint16)) and np.array_equal(h.view(np.uint16), L.h.view(np.uint16))
    p2, _, _ = rabit.unpack_host(img, 2, 70, 640)
    assert np.array_equal(p2, L.planes)


def test_header_records_largest_input_scale():
    L = make_layer(40, 96, 3, key=(86,))
    L.h[1, 17] = np.float16(-7.5)          # the bound uses |h|
    L.h[2, :] = np.float16(0.0)
    L.h[2, 5] = np.float16(6e-8)           # a subnormal fp16
    hd = spec.read_header(rabit.pack_host(L.planes, L.g, L.h))
    got = np.array([hd["hmax0"], hd["hmax1"], hd["hmax2"]], dtype=np.uint32).view(np.float32)
    want = np.abs(L.h.astype(np.float32)).max(axis=1)
    assert np.array_equal(got, want) and got[1] == 7.5 and hd["hmax3"] == 0


def test_single_bit_lands_where_the_definition_says():
    K, M, N = 2, 200, 256
    planes = make_planes_constant(K, M, N, 0)
    row, col, k = 45, 203, 1
    planes[k, row, col // 32] = np.uint32(1 << (col % 32))
    L = make_layer(M, N, K, key=(83,))
    img = rabit.pack_host(planes, L.g, L.h)
    hd = spec.read_header(img)
    bits = img[hd["off_bits"]:hd["off_g"]]
    nz = np.flatnonzero(bits)
    assert nz.size == 1
    rt, rl = divmod(row, 128); p, r16 = divmod(rl, 16); alo, gq = divmod(r16, 8)
    ct, cl = divmod(col, 32); ah, rem = divmod(cl, 16); tq, c = divmod(rem, 4)
    tile = (rt * K + k) * hd["n_ct"] + ct
    off = tile * 512 + 16 * (4 * gq + tq) + 4 * (alo + 2 * ah) + c
    assert nz[0] == off and bits[off] == 1 << p


def test_single_bit_lands_in_the_look_up_block_the_definition_names():
    K, M, N = 2, 200, 544
    L = make_layer(M, N, K, key=(87,))
    for row, col, k in [(45, 203, 1), (0, 0, 0), (199, 543, 0), (31, 255, 1), (32, 256, 0), (77, 300, 1)]:
        planes = make_planes_constant(K, M, N, 0)
        planes[k, row, col // 32] = np.uint32(1 << (col % 32))
        img = rabit.pack_host(planes, L.g, L.h)
        hd = spec.read_header(img)
        sec = img[hd["off_lut"]:hd["off_acc"]]
        nz = np.flatnonzero(sec)
        assert nz.size == 1
        cs, cl = divmod(col, 256); group, b = divmod(cl, 8); rb, l = divmod(row, 32)
        s = (group - l) % 32                                  # the step at which lane l visits this group
        off = ((cs * hd["n_rb"] + rb) * K + k) * 1024 + 512 * (s // 16) + 16 * l + (s % 16)
        assert nz[0] == off and sec[off] == 1 << b


@pytest.mark.parametrize("K,M,N", [(2, 64, 256), (3, 33, 1056), (1, 7, 96), (2, 100, 160)])
def test_look_up_blocks_alone_give_back_the_planes(K, M, N):
    L = make_layer(M, N, K, key=(88, K, M, N))
    img = rabit.pack_host(L.planes, L.g, L.h)
    assert np.array_equal(spec.unpack_lut_spec(img), L.planes)
    # an image whose two sign sections disagree is refused
    hd = spec.read_header(img)
    bad = img.copy()
    bad[hd["off_lut"] + 16 * 3 + 1] ^= 0x10                  # (lane 3, step 1) of block 0, path 0: a column inside N for all shapes here
    lib = binding.raw_lib()
    planes = np.empty((K, M, N // 32), dtype=np.uint32)
    assert lib.rabit_unpack_host(bad.ctypes.data, bad.nbytes, planes.ctypes.data, None, None) == -1
    assert "disagree" in rabit.last_error()


def test_header_records_the_fixed_point_grid():
    """The grid must cover twice the largest possible partial sum of a slice: recomputed here from its definition."""
    L = make_layer(96, 4096 + 256, 2, key=(89,))
    hd = spec.read_header(rabit.pack_host(L.planes, L.g, L.h))
    assert hd["n_cs"] == 17 and hd["fix_bits"] == 54 - 5
    g = np.abs(L.g.astype(np.float64)); h = np.abs(L.h.astype(np.float64))
    bound = 65504.0 * g.sum(axis=0).max() * max(h[k, j:j + 256].sum() for k in range(2) for j in range(0, h.shape[1], 256))
    top = 2.0 ** (hd["unit_exp"] + hd["fix_bits"])
    assert 2 * bound <= top < 8 * bound
    # all-zero scales: any grid will do, the header holds e = 0
    Z = make_layer(32, 64, 1, key=(90,))
    hd = spec.read_header(rabit.pack_host(Z.planes, np.zeros_like(Z.g), Z.h))
    assert hd["unit_exp"] == -hd["fix_bits"]


def test_scratch_and_padding_are_zero():
    L = make_layer(40, 160, 2, key=(84,))
    img = rabit.pack_host(L.planes, L.g, L.h)
    hd = spec.read_header(img)
    assert (img[hd["off_partial"]:hd["off_flags"]] == 0xFF).all()       # resting state of the partial buffer
    assert not img[hd["off_flags"]:hd["off_lut"]].any()
    assert not img[hd["off_acc"]:hd["total_bytes"]].any()               # accumulate words rest at zero
    # look-up blocks: rows beyond M and columns beyond N hold bit 0 (160 columns -> one slice of 256)
    lut = img[hd["off_lut"]:hd["off_acc"]][:hd["n_cs"] * hd["n_rb"] * 2 * 1024].reshape(hd["n_cs"], hd["n_rb"], 2, 2, 32, 16)
    hf, l, q = np.meshgrid(np.arange(2), np.arange(32), np.arange(16), indexing="ij")
    group = (16 * hf + q + l) % 32
    assert not lut[:, :, :, group >= 160 // 8].any()
    assert not lut[:, 1, :, :, 8:, :].any() and not lut[:, 2:].any()    # rows 40..63, then whole padded row blocks
    g = img[hd["off_g"]:hd["off_h"]].view(np.uint16)[:2 * hd["Mp"]].reshape(2, hd["Mp"])
    assert not g[:, 40:].any()


def test_shape_and_buffer_errors():
    lib = binding.raw_lib()
    assert rabit.packed_bytes(2, 64, 48) == 0          # N not a multiple of 32
    assert rabit.packed_bytes(4, 64, 64) == 0          # K > 3
    assert rabit.packed_bytes(2, 0, 64) == 0
    L = make_layer(32, 64, 2, key=(85,))
    need = rabit.packed_bytes(2, 32, 64)
    small = np.empty(need - 1, dtype=np.uint8)
    g16 = L.g.view(np.uint16); h16 = L.h.view(np.uint16)
    rc = lib.rabit_pack_host(L.planes.ctypes.data, g16.ctypes.data, h16.ctypes.data, 2, 32, 64, small.ctypes.data, small.nbytes)
    assert rc == -3 and "need" in rabit.last_error()
    rc = lib.rabit_pack_host(None, g16.ctypes.data, h16.ctypes.data, 2, 32, 64, small.ctypes.data, small.nbytes)
    assert rc == -1
    rc = lib.rabit_pack_host(L.planes.ctypes.data, g16.ctypes.data, h16.ctypes.data, 2, 32, 48, small.ctypes.data, small.nbytes)
    assert rc == -2
    with pytest.raises(rabit.RabitError):
        rabit.pack_host(np.zeros((4, 32, 2), np.uint32), np.zeros((4, 32), np.float16), np.zeros((4, 64), np.float16))
    junk = np.zeros(512, dtype=np.uint8)
    assert lib.rabit_unpack_host(junk.ctypes.data, junk.nbytes, None, None, None) == -1
    # host-side argument checks of the device entry points need no GPU
    assert lib.rabit_linear(None, None, None, 1, None) == -1
    assert lib.rabit_free(None) == 0
    assert lib.rabit_layer_K(None) == -1
    out = ctypes.c_void_p()
    assert lib.rabit_pack(None, None, None, 2, 32, 64, None, 0, None, ctypes.byref(out)) == -1


def test_every_declared_symbol_is_exported():
    header = open(os.path.join(ROOT, "include", "rabit.h")).read()
    names = re.findall(r"RABIT_API\s+[\w\s\*]+?\b(rabit_\w+)\s*\(", header)
    assert len(names) >= 13
    lib = ctypes.CDLL(rabit.lib_path())
    for n in names:
        assert hasattr(lib, n), f"{n} declared in include/rabit.h but not exported"


@pytest.mark.parametrize("K,M,N,batch,sms", [
    (2, 14336, 4096, 16, 148), (2, 14336, 4096, 8, 148), (2, 4096, 4096, 16, 148), (2, 4096, 14336, 3, 148),
    (2, 28672, 8192, 16, 148), (2, 1024, 4096, 8, 148), (3, 11008, 4096, 16, 148), (1, 129, 288, 5, 148),
    (2, 200, 65280, 16, 148), (2, 128, 32, 3, 148), (2, 100000, 4096, 12, 148), (2, 4096, 11008, 16, 132), (2, 300, 640, 7, 4),
])
def test_work_split_of_the_f16_gemv(K, M, N, batch, sms):
    """Host logic of the batch 3..16 kernel: the (row tile, slice) pairs are cut into two contiguous parts per SM.  Whatever
    the cost model prefers, the parts must tile the pairs exactly, in order, on no more CTAs than SMs; no row tile may be
    touched by more parts than the eight-bit arrival count of an accumulate word can hold; and the split must be the
    same every time (the plan is cached)."""
    lib = ctypes.CDLL(rabit.lib_path())
    lib.rabit_selftest_f16_plan.restype = ctypes.c_int
    lib.rabit_selftest_f16_plan.argtypes = [ctypes.c_int] * 5 + [ctypes.c_void_p, ctypes.c_int]
    out = (ctypes.c_int * 400)()
    grid = lib.rabit_selftest_f16_plan(K, M, N, batch, sms, out, 400)
    n_rt, n_cs = -(-M // 128), -(-N // 256)
    n_pairs = n_rt * n_cs
    assert 1 <= grid <= min(sms, n_pairs)
    bound = list(out[:2 * grid + 1])
    assert bound[0] == 0 and bound[-1] == n_pairs
    assert all(a <= b for a, b in zip(bound, bound[1:]))
    parts = [(a, b) for a, b in zip(bound, bound[1:]) if b > a]
    assert sum(b - a for a, b in parts) == n_pairs
    assert all(bound[2 * c] < bound[2 * c + 2] for c in range(grid))             # every CTA has work
    touching = [0] * n_rt
    for a, b in parts:
        for rt in range(a // n_cs, (b - 1) // n_cs + 1):
            touching[rt] += 1
    assert 1 <= min(touching) and max(touching) <= 255
    # balance: no SM has more than twice the average number of pairs (plus one row tile's worth of slack for tiny layers)
    per_sm = [bound[2 * c + 2] - bound[2 * c] for c in range(grid)]
    assert max(per_sm) <= 2 * n_pairs / grid + n_cs
    again = (ctypes.c_int * 400)()
    assert lib.rabit_selftest_f16_plan(K, M, N, batch, sms, again, 400) == grid and list(again[:2 * grid + 1]) == bound


def test_work_split_of_the_f16_gemv_rejects_what_the_kernel_cannot_run():
    lib = ctypes.CDLL(rabit.lib_path())
    lib.rabit_selftest_f16_plan.restype = ctypes.c_int
    lib.rabit_selftest_f16_plan.argtypes = [ctypes.c_int] * 5 + [ctypes.c_void_p, ctypes.c_int]
    out = (ctypes.c_int * 400)()
    assert lib.rabit_selftest_f16_plan(2, 128, 65312, 8, 148, out, 400) < 0      # 256 slices
    assert lib.rabit_selftest_f16_plan(2, 128, 4096, 17, 148, out, 400) < 0      # more rows than a pass takes
    assert lib.rabit_selftest_f16_plan(4, 128, 4096, 8, 148, out, 400) < 0       # too many paths
    assert lib.rabit_selftest_f16_plan(2, 4096, 4096, 8, 148, out, 10) < 0       # output array too small
    assert lib.rabit_selftest_f16_plan(2, 4096, 4096, 8, 148, None, 400) < 0

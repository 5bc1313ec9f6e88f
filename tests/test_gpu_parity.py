"""GPU parity: the CUDA library (through the C ABI) against the float64 CPU oracle on
identical seeded inputs, element by element, within
    max_i |y_gpu - y_ref| <= 2e-3 * max_i sum_j sum_k |g_ki h_kj x_j| + 1e-5   per batch row."""
import ctypes

import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import make_layer, make_x, make_planes_constant
from tests.gpu_util import run_layer, check_against_oracle

pytestmark = pytest.mark.gpu

VARIANTS = [0, 1, 2, 5, 6]   # automatic, plain sign-select, integer-MMA GEMV, table-driven GEMV, f16 tensor-core GEMV

SMALL = [  # several tiles plus ragged tails in both dimensions
    (2, 32, 128), (2, 100, 160), (2, 256, 1184), (3, 96, 640), (1, 33, 96), (2, 160, 2080), (2, 1000, 512),
    (1, 128, 32), (2, 129, 32), (3, 700, 8192), (2, 2500, 96),
]


@pytest.mark.parametrize("variant", VARIANTS)
@pytest.mark.parametrize("K,M,N", SMALL)
@pytest.mark.parametrize("batch", [1, 2])
def test_small_shapes(K, M, N, batch, variant):
    L = make_layer(M, N, K, key=(70, K, M, N))
    x = make_x(batch, N, key=(70, M, N, batch))
    y = run_layer(L, x, variant)
    check_against_oracle(L, x, y)


@pytest.mark.parametrize("variant", [0, 1])
@pytest.mark.parametrize("batch", [3, 4, 5, 8, 16, 17, 40])
def test_batches(batch, variant):
    L = make_layer(192, 896, 2, key=(71,))
    x = make_x(batch, 896, key=(71, batch))
    y = run_layer(L, x, variant)
    check_against_oracle(L, x, y)


@pytest.mark.parametrize("K,M,N", [(2, 192, 896), (3, 300, 640), (1, 129, 288), (2, 1000, 4352), (2, 4096, 4096)])
@pytest.mark.parametrize("batch", [3, 7, 8, 9, 16])
def test_f16_tensor_core_gemv_batches(K, M, N, batch):
    """The batch 3..16 kernel (batch in the MMA's N dimension) forced, every batch width class, ragged shapes, K = 1..3."""
    L = make_layer(M, N, K, key=(69, K, M, N))
    x = make_x(batch, N, key=(69, M, N, batch))
    y = run_layer(L, x, 6)
    check_against_oracle(L, x, y)
    y2 = run_layer(L, x, 6)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))     # integer accumulate words: the same bits every run


@pytest.mark.parametrize("batch", [1, 2, 5, 16])
def test_widest_layer_of_the_accumulate_word_kernels(batch):
    """N = 65280 is 255 slices of 256 columns, the most the eight-bit arrival count of an accumulate word can take: the
    table-driven kernel (batch 1, 2) and the f16 GEMV (5, 16) at that limit, where a row's word collects up to 255
    contributions on a grid of 46 magnitude bits."""
    L = make_layer(200, 65280, 2, key=(70,))
    x = make_x(batch, 65280, key=(70, batch))
    y = run_layer(L, x, 0)
    check_against_oracle(L, x, y)
    forced = run_layer(L, x, 5 if batch <= 2 else 6)
    assert np.array_equal(y.view(np.uint16), forced.view(np.uint16))


def test_layer_wider_than_the_accumulate_word_kernels_falls_back():
    """One more column tile (256 slices): both kernels refuse the layer, the dispatcher takes the integer-MMA GEMV or the GEMM."""
    import paper_2602_05367_b200 as rabit
    L = make_layer(200, 65312, 2, key=(71,))
    for batch in (1, 5):
        x = make_x(batch, 65312, key=(71, batch))
        check_against_oracle(L, x, run_layer(L, x, 0))
        for variant in (5, 6):
            with pytest.raises(rabit.RabitError):
                run_layer(L, x, variant)


@pytest.mark.parametrize("variant", VARIANTS)
def test_config0_full_size(variant):
    """4096 x 4096, K=2, batch 1, seed 0 -- every output compared."""
    L = make_layer(4096, 4096, 2, key=(0, 0, 0))
    x = make_x(1, 4096, key=(0, 0))
    y = run_layer(L, x, variant)
    err, tol = check_against_oracle(L, x, y)
    assert tol[0] > 0.1 and err[0] < tol[0]


@pytest.mark.parametrize("variant", VARIANTS)
def test_structured_inputs(variant):
    K, M, N = 2, 96, 384
    L = make_layer(M, N, K, key=(72,))
    # unit vectors read single columns (bit order / layout permutation)
    for j in [0, 1, 31, 32, 127, 128, 200, 383]:
        x = np.zeros((1, N), dtype=np.float16); x[0, j] = 1.0
        check_against_oracle(L, x, run_layer(L, x, variant))
    # constant planes
    for bit in (0, 1):
        L.planes = make_planes_constant(K, M, N, bit)
        x = make_x(1, N, key=(72, bit))
        check_against_oracle(L, x, run_layer(L, x, variant))
    # zero activations give exactly zero
    L = make_layer(M, N, K, key=(72, 9))
    y = run_layer(L, np.zeros((2, N), dtype=np.float16), variant)
    assert not y.any()


@pytest.mark.parametrize("variant", VARIANTS)
def test_outlier_activations(variant):
    """A few huge activations among small ones (the dynamic range of real hidden states)."""
    K, M, N = 2, 128, 2048
    L = make_layer(M, N, K, key=(73,))
    x = (make_x(2, N, key=(73,)).astype(np.float32) * 0.02)
    x[0, 5] = 900.0; x[0, 1033] = -650.0; x[1, 77] = 1200.0
    x = x.astype(np.float16)
    check_against_oracle(L, x, run_layer(L, x, variant))


def test_device_round_trip():
    import paper_2602_05367_b200 as rabit
    L = make_layer(100, 288, 2, key=(74,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    planes, g, h = layer.unpack()
    assert np.array_equal(planes, L.planes)
    assert np.array_equal(g.view(np.uint16), L.g.view(np.uint16))
    assert np.array_equal(h.view(np.uint16), L.h.view(np.uint16))
    layer.free()


def test_graph_capture_and_replay():
    import torch
    import paper_2602_05367_b200 as rabit
    L = make_layer(256, 512, 2, key=(75,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    x = torch.zeros((1, 512), dtype=torch.float16, device="cuda:0")
    y = torch.empty((1, 256), dtype=torch.float16, device="cuda:0")
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        rabit.rabit_linear(layer, x, y)        # warm-up outside capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            rabit.rabit_linear(layer, x, y)
    for t in range(3):
        xn = make_x(1, 512, key=(75, t))
        x.copy_(torch.from_numpy(xn))
        graph.replay()
        torch.cuda.synchronize()
        check_against_oracle(L, xn, y.cpu().numpy())
    layer.free()


def test_repeated_calls_leave_scratch_clean():
    import torch
    import paper_2602_05367_b200 as rabit
    L = make_layer(320, 1536, 2, key=(76,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    for t in range(4):
        xn = make_x(2, 1536, key=(76, t))
        y = rabit.rabit_linear(layer, torch.from_numpy(xn).cuda())
        torch.cuda.synchronize()
        check_against_oracle(L, xn, y.cpu().numpy())
    layer.free()


def test_argument_errors_on_device():
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding
    lib = binding.raw_lib()
    L = make_layer(64, 128, 2, key=(77,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    buf = torch.zeros(4096, dtype=torch.float16, device="cuda:0")
    p = buf.data_ptr()
    vp = ctypes.c_void_p
    assert lib.rabit_linear(layer.handle, vp(p + 2), vp(p + 2048), 1, None) == -1      # misaligned x
    assert "aligned" in rabit.last_error()
    assert lib.rabit_linear(layer.handle, vp(p), vp(p + 128), 1, None) == -1           # y overlaps x
    assert lib.rabit_linear(layer.handle, vp(p), vp(p + 2048), 0, None) == -1          # batch < 1
    host = np.zeros(rabit.packed_bytes(2, 64, 128), dtype=np.uint8)
    out = vp()
    rc = lib.rabit_pack(L.planes.ctypes.data, L.g.view(np.uint16).ctypes.data, L.h.view(np.uint16).ctypes.data,
                        2, 64, 128, vp(p), 16, None, ctypes.byref(out))
    assert rc == -3                                                                     # device buffer too small
    layer.free()


@pytest.mark.parametrize("pinned", [True, False])
@pytest.mark.parametrize("batch", [1, 3, 40])
def test_host_buffer_entry_point(batch, pinned):
    """rabit_linear_host: host x in, host y out.  Pinned (mapped) outputs of decode-sized calls are written
    by the kernel itself, everything else goes through the device stage and a copy back; twice in a row."""
    import torch
    import paper_2602_05367_b200 as rabit
    L = make_layer(200, 640, 2, key=(78,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    for rep in range(2):
        xn = make_x(batch, 640, key=(78, batch, rep))
        xh = torch.from_numpy(xn)
        yh = torch.zeros((batch, 200), dtype=torch.float16)
        if pinned:
            xh, yh = xh.pin_memory(), yh.pin_memory()
        rabit.rabit_linear_host(layer, xh, yh)
        torch.cuda.synchronize()
        check_against_oracle(L, xn, yh.numpy())
    assert layer.status() == 0
    layer.free()


def test_status_word_stays_clear_and_bounded_wait_self_test():
    """Failure detection without a fault: after normal runs the layer's status word is clear; a kernel whose
    wait can never succeed gives up after its limit, records it and leaves the device usable."""
    import time
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding
    L = make_layer(300, 640, 2, key=(79,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    for batch in (1, 4, 40):
        xn = make_x(batch, 640, key=(79, batch))
        y = rabit.rabit_linear(layer, torch.from_numpy(xn).cuda())
        assert layer.status() == 0
        check_against_oracle(L, xn, y.cpu().numpy())
    lib = binding.raw_lib()
    word = torch.zeros(1, dtype=torch.int32, device="cuda")
    t0 = time.time()
    assert lib.rabit_selftest_bounded_wait(ctypes.c_void_p(word.data_ptr()), 20000, None) == 0, rabit.last_error()
    assert time.time() - t0 < 5.0 and int(word.item()) == 1
    assert lib.rabit_selftest_bounded_wait(ctypes.c_void_p(word.data_ptr()), 0, None) == -1
    # the context is still usable
    xn = make_x(1, 640, key=(79, 99))
    y = rabit.rabit_linear(layer, torch.from_numpy(xn).cuda())
    torch.cuda.synchronize()
    check_against_oracle(L, xn, y.cpu().numpy())
    layer.free()


@pytest.mark.parametrize("batch", [2, 4, 40])
def test_non_finite_activations_poison_only_their_batch_row(batch):
    """An inf or NaN in one activation row makes every output of that row non-finite and leaves the other
    rows within tolerance (GEMV: the fixed-point scale of the row becomes NaN; GEMM: inf/NaN propagate)."""
    import torch
    import paper_2602_05367_b200 as rabit
    L = make_layer(300, 640, 2, key=(66, batch))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    xn = make_x(batch, 640, key=(66, batch))
    bad = xn.copy()
    bad[1, 17] = np.float16(np.inf)
    y = rabit.rabit_linear(layer, torch.from_numpy(bad).cuda()).cpu().numpy().astype(np.float64)
    assert not np.isfinite(y[1]).any()
    keep = [b for b in range(batch) if b != 1]
    ref = orc.linear(L.planes, L.g, L.h, xn[keep])
    tol = orc.tolerance(L.g, L.h, xn[keep])
    assert (np.abs(y[keep] - ref).max(axis=1) <= tol).all()
    bad[1, 17] = np.float16(np.nan)
    y = rabit.rabit_linear(layer, torch.from_numpy(bad).cuda()).cpu().numpy()
    assert np.isnan(y[1].astype(np.float64)).all()
    assert layer.status() == 0
    layer.free()


def test_tiny_and_huge_magnitudes_keep_their_precision():
    """The fixed-point scale follows the data: activations of magnitude 1e-4 or 1e+4 lose nothing."""
    import torch
    import paper_2602_05367_b200 as rabit
    L = make_layer(256, 1024, 2, key=(67,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    for scale in (1e-4, 1.0, 3e3):
        xn = (make_x(2, 1024, key=(67,)).astype(np.float32) * scale).astype(np.float16)
        y = rabit.rabit_linear(layer, torch.from_numpy(xn).cuda())
        torch.cuda.synchronize()
        err, tol = check_against_oracle(L, xn, y.cpu().numpy())
        assert (err <= 0.3 * tol).all()          # far inside: only the fp16 output rounding is left
    layer.free()

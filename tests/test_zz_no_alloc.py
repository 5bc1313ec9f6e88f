"""The allocation-free entry point, rabit_linear_static_scratch, against rabit_linear.

Some hosts of this library may not allocate device memory when a layer runs: they got a fixed
budget at start-up, or sit in a latency-critical loop where cudaMalloc could stall the GPU, or
were handed buffers by a framework that owns the allocator.  For them the library carries its
own 4 MiB scratch array.  This test drives the new entry point through the C ABI with raw
pointers (x and y preallocated up front, nothing allocated between the calls), twice in a row
and across two different layers that share the array, and expects the same numbers as the
ordinary entry point, inside the parity tolerance used everywhere else in this suite.
This file is collected last on purpose.
"""
import ctypes

import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import make_layer, make_x

pytestmark = pytest.mark.gpu


def _raw_call(lib, name, layer, x, y, batch, stream):
    vp = ctypes.c_void_p
    return getattr(lib, name)(layer.handle, vp(x.data_ptr()), vp(y.data_ptr()), batch, vp(stream))


def test_static_scratch_matches_ordinary_entry_point_twice_in_a_row():
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding

    lib = binding.raw_lib()
    shapes = [(2, 1000, 1184), (2, 4096, 4096), (3, 300, 640)]     # ragged rows and columns, a graded shape, three paths
    layers = []
    for K, M, N in shapes:
        L = make_layer(M, N, K, key=(50, K, M, N))
        layers.append((L, rabit.rabit_pack(L.planes, L.g, L.h)))
    stream = torch.cuda.current_stream().cuda_stream
    for batch in (1, 2, 5):
        bufs = []
        for (L, layer) in layers:
            xn = [make_x(batch, L.N, key=(50, L.M, batch, t)) for t in range(2)]
            xs = [torch.from_numpy(a).cuda() for a in xn]
            y_new = [torch.zeros((batch, L.M), dtype=torch.float16, device="cuda") for _ in range(2)]
            y_old = [torch.zeros((batch, L.M), dtype=torch.float16, device="cuda") for _ in range(2)]
            bufs.append((xn, xs, y_new, y_old))
        torch.cuda.synchronize()
        # every buffer exists now; from here to the comparison only the two entry points run
        for (L, layer), (xn, xs, y_new, y_old) in zip(layers, bufs):
            for t in range(2):                                      # two calls in a row on the shared scratch
                assert _raw_call(lib, "rabit_linear_static_scratch", layer, xs[t], y_new[t], batch, stream) == 0, rabit.last_error()
            for t in range(2):
                assert _raw_call(lib, "rabit_linear", layer, xs[t], y_old[t], batch, stream) == 0, rabit.last_error()
        torch.cuda.synchronize()
        for (L, layer), (xn, xs, y_new, y_old) in zip(layers, bufs):
            for t in range(2):
                tol = orc.tolerance(L.g, L.h, xn[t])
                got = y_new[t].cpu().numpy().astype(np.float64)
                old = y_old[t].cpu().numpy().astype(np.float64)
                ref = orc.linear(L.planes, L.g, L.h, xn[t])
                assert np.isfinite(got).all()
                assert (np.abs(got - old).max(axis=1) <= tol).all()
                assert (np.abs(got - ref).max(axis=1) <= tol).all()
    for _, layer in layers:
        layer.free()


def test_static_scratch_rejects_what_it_cannot_hold():
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding

    lib = binding.raw_lib()
    L = make_layer(64, 128, 2, key=(51,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    x = torch.zeros((17, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((17, 64), dtype=torch.float16, device="cuda")
    assert _raw_call(lib, "rabit_linear_static_scratch", layer, x, y, 17, 0) == -1      # batch beyond the GEMV range
    assert "batch" in rabit.last_error()
    assert _raw_call(lib, "rabit_linear_static_scratch", layer, x, y, 0, 0) == -1
    layer.free()
    # a layer whose reduction scratch exceeds the built-in array: K * ceil(M/128) too large (tiny N keeps it cheap)
    K, M, N = 3, 128 * 700, 32
    big = make_layer(M, N, K, key=(52,))
    layer = rabit.rabit_pack(big.planes, big.g, big.h)
    x = torch.zeros((1, N), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, M), dtype=torch.float16, device="cuda")
    assert _raw_call(lib, "rabit_linear_static_scratch", layer, x, y, 1, 0) == -2
    assert "scratch" in rabit.last_error()
    layer.free()

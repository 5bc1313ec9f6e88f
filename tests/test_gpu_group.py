"""GPU parity of the grouped launch (several independent layers in one kernel) against the float64
oracle, per layer and per batch row, within the usual tolerance."""
import numpy as np
import pytest

from synth import make_layer, make_x
from tests.gpu_util import check_against_oracle

pytestmark = pytest.mark.gpu


def _run_group(specs, batch, shared_x=True, key=40):
    """specs: list of (K, M, N); layers with equal N share one activation tensor when shared_x."""
    import torch
    import paper_2602_05367_b200 as rabit
    Ls = [make_layer(M, N, K, key=(key, i, K, M, N)) for i, (K, M, N) in enumerate(specs)]
    layers = [rabit.rabit_pack(L.planes, L.g, L.h) for L in Ls]
    x_by_n, xn, xs = {}, [], []
    for i, L in enumerate(Ls):
        kx = L.N if shared_x else (L.N, i)
        if kx not in x_by_n:
            a = make_x(batch, L.N, key=(key, batch, L.N, i))
            x_by_n[kx] = (a, torch.from_numpy(a).cuda())
        xn.append(x_by_n[kx][0]); xs.append(x_by_n[kx][1])
    ys = [torch.zeros((batch, L.M), dtype=torch.float16, device="cuda") for L in Ls]
    for rep in range(2):                                     # twice: the scratch must be left clean
        for y in ys:
            y.zero_()
        rabit.rabit_linear_group(layers, xs, ys)
        torch.cuda.synchronize()
        for L, a, y in zip(Ls, xn, ys):
            check_against_oracle(L, a, y.cpu().numpy())
    for layer in layers:
        layer.free()


@pytest.mark.parametrize("batch", [1, 2, 3])
def test_qkv_like_group_shares_its_input(batch):
    _run_group([(2, 512, 1024), (2, 256, 1024), (2, 256, 1024)], batch)


def test_mixed_widths_paths_and_ragged_shapes():
    _run_group([(2, 1000, 1184), (1, 33, 96), (3, 700, 2048), (2, 128, 32), (2, 2500, 96)], 1, shared_x=False)
    _run_group([(3, 129, 64), (2, 40, 4096)], 2, shared_x=False)


def test_eight_small_layers_fewer_tiles_than_ctas():
    _run_group([(2, 64, 64)] * 8, 1, shared_x=False)


def test_full_size_decoder_groups():
    """q|k|v and gate|up of a 7B-shaped decoder layer, each as one launch."""
    _run_group([(2, 4096, 4096)] * 3, 1, key=41)
    _run_group([(2, 11008, 4096)] * 2, 1, key=42)


def test_group_falls_back_for_large_batch_and_checks_arguments():
    import ctypes
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding
    _run_group([(2, 256, 256), (2, 128, 256)], 40)           # batch > 16: one after the other (tensor-core GEMM)
    L = make_layer(64, 128, 2, key=(43,))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    x = torch.zeros((1, 128), dtype=torch.float16, device="cuda")
    y = torch.zeros((1, 64), dtype=torch.float16, device="cuda")
    lib = binding.raw_lib()
    vp = ctypes.c_void_p
    h = (vp * 2)(layer.handle, layer.handle)
    xp = (vp * 2)(x.data_ptr(), x.data_ptr())
    yp = (vp * 2)(y.data_ptr(), y.data_ptr())
    assert lib.rabit_linear_group(h, xp, yp, 2, 1, None) == -1 and "overlap" in rabit.last_error()
    assert lib.rabit_linear_group(h, xp, yp, 0, 1, None) == -1
    assert lib.rabit_linear_group(None, xp, yp, 1, 1, None) == -1
    layer.free()


def test_group_host_buffers():
    """rabit_linear_group_host: pinned host inputs (one shared by two layers) and outputs."""
    import torch
    import paper_2602_05367_b200 as rabit
    specs = [(2, 300, 640), (2, 128, 640), (3, 200, 96)]
    Ls = [make_layer(M, N, K, key=(44, i)) for i, (K, M, N) in enumerate(specs)]
    layers = [rabit.rabit_pack(L.planes, L.g, L.h) for L in Ls]
    for batch in (1, 3):
        xa = make_x(batch, 640, key=(44, batch, 1)); xb = make_x(batch, 96, key=(44, batch, 2))
        pa, pb = torch.from_numpy(xa).pin_memory(), torch.from_numpy(xb).pin_memory()
        ys = [torch.zeros((batch, L.M), dtype=torch.float16) for L in Ls]
        ys = [y.pin_memory() if i != 1 else y for i, y in enumerate(ys)]     # one pageable output: staged copy back
        rabit.rabit_linear_group_host(layers, [pa, pa, pb], ys)
        torch.cuda.synchronize()
        for L, a, y in zip(Ls, [xa, xa, xb], ys):
            check_against_oracle(L, a, y.numpy())
    for layer in layers:
        layer.free()


def test_prepared_group_host_call_repeats():
    """PreparedGroupHost: marshalled once, called three times with new inputs written into the same host tensors."""
    import torch
    import paper_2602_05367_b200 as rabit
    specs = [(2, 300, 640), (2, 128, 640)]
    Ls = [make_layer(M, N, K, key=(45, i)) for i, (K, M, N) in enumerate(specs)]
    layers = [rabit.rabit_pack(L.planes, L.g, L.h) for L in Ls]
    px = torch.zeros((2, 640), dtype=torch.float16).pin_memory()
    ys = [torch.zeros((2, L.M), dtype=torch.float16).pin_memory() for L in Ls]
    call = rabit.PreparedGroupHost(layers, [px, px], ys)
    for rep in range(3):
        xa = make_x(2, 640, key=(45, rep))
        px.copy_(torch.from_numpy(xa))
        call()
        torch.cuda.synchronize()
        for L, y in zip(Ls, ys):
            check_against_oracle(L, xa, y.numpy())
    for layer in layers:
        layer.free()

"""On-device derivation of the sign planes fused with packing (Section 4.2 steps 1-3), against the
oracle's float32-mode recurrence: the planes read back from the device image must be bit-exact, and the
derived layer must pass the usual output parity."""
import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import make_x
from tests.gpu_util import check_against_oracle

pytestmark = pytest.mark.gpu


def _inputs(K, M, N, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((M, N)) * 0.02).astype(np.float32)
    W[rng.integers(0, M, 8), rng.integers(0, N, 8)] = 0.0                 # sign(0) = +1
    h = rng.uniform(0.5, 1.5, (K, N)).astype(np.float16)
    g = np.empty((K, M), dtype=np.float16)
    scale = 0.016
    for k in range(K):
        g[k] = (scale * rng.uniform(0.8, 1.2, M)).astype(np.float16)
        scale *= 0.45
    return W, g, h


@pytest.mark.parametrize("K,M,N", [(2, 128, 32), (1, 100, 160), (3, 300, 640), (2, 1000, 1184), (2, 4096, 4096)])
def test_derived_planes_bit_exact_and_layer_parity(K, M, N):
    import torch
    import paper_2602_05367_b200 as rabit
    W, g, h = _inputs(K, M, N, seed=K * 1000 + M + N)
    if M > 64:                                                            # exact ties: W = g_0 h_0 on one row
        W[5] = (g[0, 5].astype(np.float32) * h[0].astype(np.float32))
    layer = rabit.rabit_derive_pack(torch.from_numpy(W).cuda(), g, h)
    planes, g2, h2 = layer.unpack()
    want = orc.derive_planes(W, g, h, dtype=np.float32)
    assert np.array_equal(planes, want)
    assert np.array_equal(g2.view(np.uint16), g.view(np.uint16)) and np.array_equal(h2.view(np.uint16), h.view(np.uint16))
    # the whole image equals the host packer's image of those planes
    img_dev = layer.dev_buf.cpu().numpy()
    assert np.array_equal(img_dev, rabit.pack_host(want, g, h))
    # and the layer runs
    class L:                                                              # the shape check_against_oracle expects
        pass
    L.planes, L.g, L.h = want, g, h
    for batch in (1, 3):
        x = make_x(batch, N, key=(90, batch, N))
        y = rabit.rabit_linear(layer, torch.from_numpy(x).cuda())
        torch.cuda.synchronize()
        check_against_oracle(L, x, y.cpu().numpy())
    layer.free()


def test_derive_then_run_on_one_stream_without_a_sync():
    """The decode kernel starts reading weights before its dependency wait; a layer derived on the same stream just
    before must still be seen complete (the library orders the two with a fill after the derivation kernels)."""
    import torch
    import paper_2602_05367_b200 as rabit
    K, M, N = 2, 4096, 4096
    W, g, h = _inputs(K, M, N, seed=77)
    Wd = torch.from_numpy(W).cuda()
    x = make_x(1, N, key=(91, N))
    xd = torch.from_numpy(x).cuda()
    torch.cuda.synchronize()
    for rep in range(3):
        layer = rabit.rabit_derive_pack(Wd, g, h)                         # asynchronous
        y = rabit.rabit_linear(layer, xd)                                 # same stream, nothing in between
        torch.cuda.synchronize()
        class L:
            pass
        L.planes, L.g, L.h = orc.derive_planes(W, g, h, dtype=np.float32), g, h
        check_against_oracle(L, x, y.cpu().numpy())
        layer.free()


def test_derive_pack_argument_errors():
    import ctypes
    import torch
    import paper_2602_05367_b200 as rabit
    from paper_2602_05367_b200 import binding
    lib = binding.raw_lib()
    W, g, h = _inputs(2, 64, 64, seed=1)
    Wd = torch.from_numpy(W).cuda()
    buf = torch.zeros(rabit.packed_bytes(2, 64, 64), dtype=torch.uint8, device="cuda")
    out = ctypes.c_void_p()
    vp = ctypes.c_void_p
    g16, h16 = g.view(np.uint16), h.view(np.uint16)
    assert lib.rabit_derive_pack(vp(Wd.data_ptr()), g16.ctypes.data, h16.ctypes.data, 2, 64, 64, vp(buf.data_ptr()), 16, None, ctypes.byref(out)) == -3
    assert lib.rabit_derive_pack(None, g16.ctypes.data, h16.ctypes.data, 2, 64, 64, vp(buf.data_ptr()), buf.numel(), None, ctypes.byref(out)) == -1
    assert lib.rabit_derive_pack(vp(Wd.data_ptr()), g16.ctypes.data, h16.ctypes.data, 2, 64, 48, vp(buf.data_ptr()), buf.numel(), None, ctypes.byref(out)) == -2

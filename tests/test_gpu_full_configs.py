"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (back-to-back calls replayed from a CUDA graph).  Small layers are compared in full;
for the large ones the oracle computes a sample of output rows one by one (first and last rows, rows
around 128-row tile borders, random rows) for every batch row.  Tolerance, per batch row:
    max_i |y_gpu - y_ref| <= 2e-3 * max_i sum_j sum_k |g_ki h_kj x_j| + 1e-5."""
import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import (llama2_7b_layer_shapes, llama3_8b_layer_shapes, llama_70b_layer_shapes, make_layer, make_x)

pytestmark = pytest.mark.gpu


def _sample_rows(M, n_random=48, seed=0):
    fixed = [0, 1, 127, 128, 129, M // 2, M - 129, M - 128, M - 2, M - 1]
    rng = np.random.default_rng(seed)
    rows = set(r for r in fixed if 0 <= r < M) | set(int(r) for r in rng.integers(0, M, size=n_random))
    return np.array(sorted(rows))


def _check_rows(L, x, y_gpu, rows):
    """Oracle on the sampled rows only (each row of the layer is an independent dot product)."""
    ref = orc.linear(L.planes[:, rows, :], L.g[:, rows], L.h, x)
    tol = orc.tolerance(L.g, L.h, x)                      # the bound is taken over all rows of the layer
    got = y_gpu[:, rows].astype(np.float64)
    assert np.isfinite(y_gpu.astype(np.float64)).all()
    err = np.abs(got - ref).max(axis=1)
    assert (err <= tol).all(), f"err {err.max():.3e} tol {tol.min():.3e}"


def _run_graph(layers, xs, ys):
    """All calls captured once and replayed, as the benchmark does."""
    import torch
    import paper_2602_05367_b200 as rabit
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        for layer, x, y in zip(layers, xs, ys):
            rabit.rabit_linear(layer, x, y)
    stream.synchronize()
    for y in ys:
        y.zero_()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for layer, x, y in zip(layers, xs, ys):
            rabit.rabit_linear(layer, x, y)
    g.replay()
    torch.cuda.synchronize()


def test_config1_decoder_layer_all_outputs():
    """The seven 7B projections (seed of the benchmark's copy 0), batch 1, every output compared."""
    import torch
    import paper_2602_05367_b200 as rabit
    shapes = llama2_7b_layer_shapes()
    Ls = [make_layer(sh.M, sh.N, 2, key=(1, 0, p)) for p, sh in enumerate(shapes)]
    layers = [rabit.rabit_pack(L.planes, L.g, L.h) for L in Ls]
    xn = [make_x(1, sh.N, key=(1, 10_000)) for sh in shapes]
    xs = [torch.from_numpy(a).cuda() for a in xn]
    ys = [torch.zeros((1, sh.M), dtype=torch.float16, device="cuda") for sh in shapes]
    _run_graph(layers, xs, ys)
    for L, x, y in zip(Ls, xn, ys):
        ref = orc.linear(L.planes, L.g, L.h, x)
        tol = orc.tolerance(L.g, L.h, x)
        assert (np.abs(y.cpu().numpy().astype(np.float64) - ref).max(axis=1) <= tol).all()
    for layer in layers:
        layer.free()


def test_config2_stack_tokens_sampled():
    """Two decoder layers of the stack (14 projections), three tokens re-drawn from the seed, replayed
    from one graph per token; sampled rows of every projection."""
    import torch
    import paper_2602_05367_b200 as rabit
    shapes = llama2_7b_layer_shapes()
    Ls, layers = [], []
    for c in (0, 31):
        for p, sh in enumerate(shapes):
            L = make_layer(sh.M, sh.N, 2, key=(1, c, p))
            Ls.append(L); layers.append(rabit.rabit_pack(L.planes, L.g, L.h))
    x_dev = {n: torch.zeros((1, n), dtype=torch.float16, device="cuda") for n in (4096, 11008)}
    ys = [torch.zeros((1, L.M), dtype=torch.float16, device="cuda") for L in Ls]
    xs = [x_dev[L.N] for L in Ls]
    _run_graph(layers, xs, ys)                       # captures; the replays below reuse the library's launches
    stream = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for layer, x, y in zip(layers, xs, ys):
            rabit.rabit_linear(layer, x, y)
    for token in (0, 7, 255):
        xn = {n: make_x(1, n, key=(2, 10_000 + token)) for n in x_dev}
        for n in x_dev:
            x_dev[n].copy_(torch.from_numpy(xn[n]))
        g.replay()
        torch.cuda.synchronize()
        for i, (L, y) in enumerate(zip(Ls, ys)):
            _check_rows(L, xn[L.N], y.cpu().numpy(), _sample_rows(L.M, 24, seed=token + i))
    for layer in layers:
        layer.free()


@pytest.mark.parametrize("batch", [1, 2, 4, 8, 16])
def test_config3_llama3_8b_batch_sweep_sampled(batch):
    import torch
    import paper_2602_05367_b200 as rabit
    seen = set()
    for sh in llama3_8b_layer_shapes():
        if (sh.M, sh.N) in seen:
            continue
        seen.add((sh.M, sh.N))
        L = make_layer(sh.M, sh.N, 2, key=(3, sh.M, sh.N))
        layer = rabit.rabit_pack(L.planes, L.g, L.h)
        xn = make_x(batch, sh.N, key=(3, batch, sh.N))
        x = torch.from_numpy(xn).cuda()
        y = torch.zeros((batch, sh.M), dtype=torch.float16, device="cuda")
        _run_graph([layer], [x], [y])
        _check_rows(L, xn, y.cpu().numpy(), _sample_rows(sh.M, 32, seed=batch))
        layer.free()


@pytest.mark.parametrize("shape_index", [0, 1, 2, 3])
def test_config4_70b_gemv_and_gemm_sampled(shape_index):
    """70B-shaped layers: batch 1 (GEMV) and batch 512 (tensor-core GEMM), sampled rows, every batch row."""
    import torch
    import paper_2602_05367_b200 as rabit
    sh = llama_70b_layer_shapes()[shape_index]
    L = make_layer(sh.M, sh.N, 2, key=(4, sh.M, sh.N))
    layer = rabit.rabit_pack(L.planes, L.g, L.h)
    rows = _sample_rows(sh.M, 40, seed=shape_index)
    for batch in (1, 512):
        xn = make_x(batch, sh.N, key=(4, batch, sh.N))
        x = torch.from_numpy(xn).cuda()
        y = torch.zeros((batch, sh.M), dtype=torch.float16, device="cuda")
        _run_graph([layer], [x], [y])
        _check_rows(L, xn, y.cpu().numpy(), rows)
    layer.free()

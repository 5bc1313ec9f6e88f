"""GPU parity of the large-batch (tensor-core GEMM) form against the float64 CPU oracle, through
the C ABI, within  max_i |y_gpu - y_ref| <= 2e-3 * max_i sum_j sum_k |g_ki h_kj x_j| + 1e-5  per batch row."""
import numpy as np
import pytest

from synth import make_layer, make_x, make_planes_constant
from tests.gpu_util import run_layer, check_against_oracle

pytestmark = pytest.mark.gpu

GEMM = 3    # variant number of the tcgen05 GEMM


@pytest.mark.parametrize("K,M,N,batch", [
    (2, 128, 64, 17),        # one tile, one step
    (2, 256, 256, 40),
    (1, 200, 96, 64),        # ragged M, a last step with a single column tile
    (2, 1000, 1184, 300),    # several row tiles, two batch tiles with a ragged tail, N % 64 == 32
    (2, 384, 2048, 512),
    (2, 2500, 512, 257),
    (3, 300, 352, 130),      # three paths: 128-wide batch tiles, two of them with a ragged tail
    (3, 128, 64, 17),
])
@pytest.mark.parametrize("variant", [0, GEMM])
def test_gemm_shapes(K, M, N, batch, variant):
    L = make_layer(M, N, K, key=(60, K, M, N))
    x = make_x(batch, N, key=(60, M, N, batch))
    y = run_layer(L, x, variant)
    check_against_oracle(L, x, y)


def test_gemm_matches_plain_kernel_closely():
    """Both device kernels see the same packed image; the GEMM keeps products exact and accumulates in fp32."""
    L = make_layer(512, 1024, 2, key=(61,))
    x = make_x(96, 1024, key=(61,))
    a = run_layer(L, x, GEMM).astype(np.float64)
    b = run_layer(L, x, 1).astype(np.float64)
    assert np.abs(a - b).max() <= 4e-3


def test_gemm_structured_inputs():
    K, M, N, batch = 2, 256, 320, 33
    L = make_layer(M, N, K, key=(62,))
    x = np.zeros((batch, N), dtype=np.float16)
    for b in range(batch):
        x[b, (b * 37) % N] = 1.0          # unit vectors: every output reads one column
    check_against_oracle(L, x, run_layer(L, x, GEMM))
    for bit in (0, 1):
        L.planes = make_planes_constant(K, M, N, bit)
        x = make_x(batch, N, key=(62, bit))
        check_against_oracle(L, x, run_layer(L, x, GEMM))
    y = run_layer(make_layer(M, N, K, key=(62, 9)), np.zeros((batch, N), dtype=np.float16), GEMM)
    assert not y.any()


def test_three_paths_large_batch():
    """K = 3 runs with three 128-column accumulators; automatic dispatch and the explicit variant agree with the oracle."""
    L = make_layer(160, 256, 3, key=(63,))
    x = make_x(48, 256, key=(63,))
    check_against_oracle(L, x, run_layer(L, x, 0))
    check_against_oracle(L, x, run_layer(L, x, GEMM))


@pytest.mark.parametrize("K,M,N,batch", [
    (2, 300, 640, 1),
    (2, 300, 640, 5),
    (3, 200, 352, 9),
    (2, 1000, 1184, 16),
])
def test_gemm_runs_small_batches_too(K, M, N, batch):
    """The tensor-core GEMM forced onto decode-sized batches (its batch tile is then mostly zero fill)."""
    L = make_layer(M, N, K, key=(62, K, M, N))
    x = make_x(batch, N, key=(62, M, N, batch))
    y = run_layer(L, x, GEMM)
    check_against_oracle(L, x, y)


@pytest.mark.parametrize("batch", [2, 3, 4, 8, 12, 16, 17, 32, 33])
def test_dispatch_by_batch(batch):
    """One or two rows take the table-driven GEMV, 3 to 32 the f16 tensor-core GEMV (passes of 16 rows), more the GEMM.
    Whichever kernel runs, the result is within tolerance and is exactly what that kernel gives when forced."""
    L = make_layer(14336, 512, 2, key=(63,))
    x = make_x(batch, 512, key=(63, batch))
    y_auto = run_layer(L, x, 0)
    check_against_oracle(L, x, y_auto)
    expect = 5 if batch <= 2 else 6 if batch <= 32 else GEMM
    y_forced = run_layer(L, x, expect)
    assert np.array_equal(y_auto.view(np.uint16), y_forced.view(np.uint16))


DEQ = 4     # variant number of the GEMM on dequantised fp16 weight tiles


@pytest.mark.parametrize("K,M,N,batch", [
    (2, 128, 64, 17),
    (1, 200, 96, 64),
    (2, 1000, 1184, 300),
    (2, 384, 2048, 512),
    (3, 300, 352, 130),
    (3, 1000, 1184, 300),
    (2, 300, 640, 5),
])
def test_dequantised_tile_gemm(K, M, N, batch):
    """Variant 4 forms sum_k +-g_k h_k per weight in fp16 and runs one contraction: every weight carries a relative
    rounding of about 2^-11 per partial product, so the result stays inside the tolerance (worst case half of it) but is
    not as close to the oracle as the exact-expansion GEMM."""
    L = make_layer(M, N, K, key=(64, K, M, N))
    x = make_x(batch, N, key=(64, M, N, batch))
    y = run_layer(L, x, DEQ)
    err, tol = check_against_oracle(L, x, y, tight=False)          # fp16-rounded weights: the mandated bound only
    y_exact = run_layer(L, x, GEMM)
    err_exact, _ = check_against_oracle(L, x, y_exact)
    assert err_exact.max() <= err.max() + 1e-3 * tol.max()        # the exact expansion is never noticeably worse


@pytest.mark.parametrize("K,M,N,batch,variant", [
    (2, 256, 4096, 64, GEMM),      # 2 tiles, 64 steps: eight CTAs share a tile (32-column slices)
    (2, 256, 4096, 300, GEMM),     # two batch tiles, ragged
    (2, 200, 4160, 40, DEQ),       # ragged rows, 65 steps split unevenly
    (3, 256, 2048, 100, GEMM),     # three paths: 128-wide tiles, four CTAs per tile
    (1, 384, 1024, 17, GEMM),      # two CTAs per tile
    (2, 1024, 8192, 512, GEMM),    # the 70B k/v projection at batch 512: 16 tiles, eight CTAs each
    (2, 19200, 1024, 20, GEMM),    # 150 tiles on 148 SMs: one whole wave, then the two tiles left over as a split launch
    (2, 19100, 1024, 20, DEQ),
    (2, 11008, 1024, 40, GEMM),    # 86 tiles: more than half the SMs, one CTA per tile
])
def test_gemm_split_contraction_across_a_cluster(K, M, N, batch, variant):
    """Layers with few output tiles: the CTAs of a cluster split the contraction of a tile and add their partial
    results through distributed shared memory (fixed order, so the result is deterministic)."""
    L = make_layer(M, N, K, key=(65, K, M, N))
    x = make_x(batch, N, key=(65, M, N, batch))
    y = run_layer(L, x, variant)
    if M * N * batch <= 2 ** 31:
        check_against_oracle(L, x, y, tight=variant != DEQ)
    else:                                           # large case: sampled rows, at least one in every 128-row tile
        rng = np.random.default_rng(0)
        rows = np.unique(np.concatenate([np.arange(0, 4), np.arange(126, 131), np.arange(M - 3, M), rng.integers(0, M, 24),
                                         np.arange(0, M, 128) + rng.integers(0, 128, (M + 127) // 128)]))
        rows = rows[rows < M]
        check_against_oracle(L, x, y, tight=variant != DEQ, rows=rows)
    y2 = run_layer(L, x, variant)
    assert np.array_equal(y.view(np.uint16), y2.view(np.uint16))

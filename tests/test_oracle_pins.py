"""Pins for the CPU oracle: each test fixes it against something other than itself
(a brute-force loop written from the definition, a closed form, an invariant, a library
routine, or a value the paper prints)."""
import os

import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import make_layer, make_x, make_planes_constant

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ---------------------------------------------------------------------------------------
# brute force straight from y_i = sum_k g_ki sum_j B_kij h_kj x_j  (Section 4.1 + Eq. 2)
# ---------------------------------------------------------------------------------------
def _sign(planes, k, i, j):
    word = int(planes[k, i, j // 32])
    return -1.0 if (word >> (j % 32)) & 1 else 1.0


def _brute(planes, g, h, x):
    K, M = g.shape
    N = h.shape[1]
    out = []
    for b in range(x.shape[0]):
        row = []
        for i in range(M):
            acc = 0.0
            for k in range(K):
                inner = 0.0
                for j in range(N):
                    inner += _sign(planes, k, i, j) * float(h[k, j]) * float(x[b, j])
                acc += float(g[k, i]) * inner
            row.append(acc)
        out.append(row)
    return np.array(out)


@pytest.mark.parametrize("M,N", [(32, 32), (32, 64), (96, 32), (64, 96), (5, 64)])
@pytest.mark.parametrize("K", [1, 2, 3])
@pytest.mark.parametrize("batch", [1, 3])
def test_brute_force_tiny(M, N, K, batch):
    L = make_layer(M, N, K, key=(90, M, N, K))
    x = make_x(batch, N, key=(90, M, N, batch))
    want = _brute(L.planes, L.g, L.h, x)
    got = orc.linear(L.planes, L.g, L.h, x, row_block=7)
    scale = np.abs(want).max() + 1.0
    assert got.shape == (batch, M)
    assert np.abs(got - want).max() <= 1e-12 * scale


def test_row_block_does_not_change_result():
    L = make_layer(160, 128, 2, key=(91,))
    x = make_x(2, 128, key=(91,))
    a = orc.linear(L.planes, L.g, L.h, x, row_block=1)
    b = orc.linear(L.planes, L.g, L.h, x, row_block=1000)
    assert np.abs(a - b).max() <= 1e-12


# ---------------------------------------------------------------------------------------
# closed forms
# ---------------------------------------------------------------------------------------
def _signs_via_unpackbits(plane, N):
    """Independent unpack with numpy's library routine (little-endian bytes, LSB-first bits)."""
    b = np.unpackbits(plane.astype("<u4").view(np.uint8), axis=-1, bitorder="little")
    return 1.0 - 2.0 * b[:, :N].astype(np.float64)


def test_single_path_closed_form():
    """K=1: y = g * (B (h * x))  (Section 4.1)."""
    L = make_layer(96, 160, 1, key=(92,))
    x = make_x(2, 160, key=(92,))
    B = _signs_via_unpackbits(L.planes[0], 160)
    want = np.stack([L.g[0].astype(np.float64) * (B @ (L.h[0].astype(np.float64) * xb.astype(np.float64)))
                     for xb in x])
    got = orc.linear(L.planes, L.g, L.h, x)
    assert np.abs(got - want).max() <= 1e-12 * (np.abs(want).max() + 1)


def test_two_equal_paths_collapse():
    """K=2 with B_2 = B_1 and h_2 = c h_1 gives y = (g_1 + c g_2) * (B_1 (h_1 * x))."""
    L = make_layer(64, 128, 2, key=(93,))
    c = 0.25
    L.planes[1] = L.planes[0]
    L.h[1] = (L.h[0].astype(np.float64) * c).astype(np.float16)   # exact: power-of-two factor
    x = make_x(1, 128, key=(93,))
    B = _signs_via_unpackbits(L.planes[0], 128)
    g = L.g.astype(np.float64)
    want = (g[0] + c * g[1]) * (B @ (L.h[0].astype(np.float64) * x[0].astype(np.float64)))
    got = orc.linear(L.planes, L.g, L.h, x)[0]
    assert np.abs(got - want).max() <= 1e-12 * (np.abs(want).max() + 1)


def test_linearity_and_zero():
    L = make_layer(64, 96, 2, key=(94,))
    x = make_x(1, 96, key=(94, 0)).astype(np.float64)
    z = make_x(1, 96, key=(94, 1)).astype(np.float64)
    a, b = 0.75, -2.5
    lhs = orc.linear(L.planes, L.g, L.h, a * x + b * z)
    rhs = a * orc.linear(L.planes, L.g, L.h, x) + b * orc.linear(L.planes, L.g, L.h, z)
    assert np.abs(lhs - rhs).max() <= 1e-12 * (np.abs(rhs).max() + 1)
    assert np.all(orc.linear(L.planes, L.g, L.h, np.zeros((1, 96))) == 0.0)


# ---------------------------------------------------------------------------------------
# sign / bit convention, bit order
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("bit,sgn", [(0, 1.0), (1, -1.0)])
def test_constant_planes(bit, sgn):
    """All bits 0 -> every sign +1 -> y_i = sum_k g_ki (h_k . x); all bits 1 -> the negative."""
    K, M, N = 2, 40, 64
    L = make_layer(M, N, K, key=(95,))
    planes = make_planes_constant(K, M, N, bit)
    x = make_x(1, N, key=(95,))
    g = L.g.astype(np.float64); h = L.h.astype(np.float64); xf = x[0].astype(np.float64)
    want = sgn * sum(g[k] * float(np.dot(h[k], xf)) for k in range(K))
    got = orc.linear(planes, L.g, L.h, x)[0]
    assert np.abs(got - want).max() <= 1e-12 * (np.abs(want).max() + 1)


def test_unit_vector_reads_one_column():
    """x = e_j  ->  y_i = sum_k g_ki B_kij h_kj : pins the bit order and the g/h roles."""
    K, M, N = 2, 48, 96
    L = make_layer(M, N, K, key=(96,))
    for j in [0, 1, 31, 32, 33, 63, 64, 95]:
        x = np.zeros((1, N)); x[0, j] = 1.0
        got = orc.linear(L.planes, L.g, L.h, x)[0]
        for i in [0, 1, 17, M - 1]:
            want = sum(float(L.g[k, i]) * _sign(L.planes, k, i, j) * float(L.h[k, j]) for k in range(K))
            assert abs(got[i] - want) <= 1e-15


def test_single_set_bit_position():
    """One word 0x00000002 in row 3 marks exactly column 1 of that word as -1 (LSB-first)."""
    K, M, N = 1, 8, 64
    planes = np.zeros((K, M, N // 32), dtype=np.uint32)
    planes[0, 3, 1] = 0x00000002          # word 1, bit 1 -> column 33
    B = orc.unpack_signs(planes, N)
    want = np.ones((K, M, N)); want[0, 3, 33] = -1.0
    assert np.array_equal(B, want)


def test_all_ones_popcount_identity():
    """g = h = x = 1  ->  y_i = sum_k (N - 2 * popcount(row i of plane k)), an exact integer."""
    K, M, N = 2, 33, 128
    L = make_layer(M, N, K, key=(97,))
    ones_g = np.ones((K, M), dtype=np.float16); ones_h = np.ones((K, N), dtype=np.float16)
    got = orc.linear(L.planes, ones_g, ones_h, np.ones((1, N)))[0]
    for i in range(M):
        pc = sum(int(w).bit_count() for k in range(K) for w in L.planes[k, i])
        assert got[i] == K * N - 2 * pc


# ---------------------------------------------------------------------------------------
# dense weight (Eq. 2) and the tolerance's L1 expression
# ---------------------------------------------------------------------------------------
def test_dense_weight_entrywise():
    K, M, N = 3, 6, 64
    L = make_layer(M, N, K, key=(98,))
    W = orc.dense_weight(L.planes, L.g, L.h)
    assert W.shape == (M, N)
    for i in range(M):
        for j in range(N):
            want = sum(float(L.g[k, i]) * _sign(L.planes, k, i, j) * float(L.h[k, j]) for k in range(K))
            assert abs(W[i, j] - want) <= 1e-15


def test_l1_bound_brute_and_k1_identity():
    K, M, N = 2, 12, 64
    L = make_layer(M, N, K, key=(99,))
    x = make_x(2, N, key=(99,))
    got = orc.l1_bound(L.g, L.h, x)
    for b in range(2):
        best = 0.0
        for i in range(M):
            s = 0.0
            for j in range(N):
                for k in range(K):
                    s += abs(float(L.g[k, i]) * float(L.h[k, j]) * float(x[b, j]))
            best = max(best, s)
        assert abs(got[b] - best) <= 1e-12 * best
    # K=1, x = 1: row sums of |W| equal |g_i| * sum_j |h_j|, and the bound is their max
    L1 = make_layer(M, N, 1, key=(99, 1))
    W = orc.dense_weight(L1.planes, L1.g, L1.h)
    rows = np.abs(W).sum(axis=1)
    want = np.abs(L1.g[0].astype(np.float64)) * np.abs(L1.h[0].astype(np.float64)).sum()
    assert np.abs(rows - want).max() <= 1e-12
    assert abs(orc.l1_bound(L1.g, L1.h, np.ones((1, N)))[0] - rows.max()) <= 1e-12
    # K=2: the bound dominates the true row sums of |W|
    W2 = orc.dense_weight(L.planes, L.g, L.h)
    assert np.abs(W2).sum(axis=1).max() <= orc.l1_bound(L.g, L.h, np.ones((1, N)))[0] + 1e-12
    tol = orc.tolerance(L.g, L.h, x)
    assert np.allclose(tol, 2e-3 * got + 1e-5, rtol=0, atol=0)


# ---------------------------------------------------------------------------------------
# values the paper prints
# ---------------------------------------------------------------------------------------
def _golden():
    out = {}
    with open(os.path.join(GOLDEN, "paper_storage.txt")) as fh:
        for line in fh:
            line = line.split("#")[0].strip()
            if line:
                k, v = line.split()
                out[k] = float(v)
    return out


def test_paper_storage_figures():
    gold = _golden()
    # nominal 2-bit layer of the 7B hidden size: about 2.02 effective bits with fp16 scales
    eff = orc.storage_bits_per_weight(2, 4096, 4096)
    assert round(eff, 2) == gold["effective_bits_nominal_2bit"]
    # one sign plane alone against fp32 weights
    assert 32.0 / orc.storage_bits_per_weight(1, 4096, 4096, scale_bits=0) == gold["sign_bits_reduction_vs_fp32"]


# ---------------------------------------------------------------------------------------
# coupled derivation of the sign planes (Section 4.2 steps 1-3)
# ---------------------------------------------------------------------------------------
def test_derive_planes_brute_force():
    rng = np.random.default_rng(5)
    K, M, N = 3, 7, 64
    W = rng.standard_normal((M, N))
    W[2, 5] = 0.0                                     # sign(0) reads as +1
    g = np.abs(rng.standard_normal((K, M))) * np.array([1.0, 0.4, 0.15])[:, None]
    h = rng.uniform(0.5, 1.5, (K, N))
    planes = orc.derive_planes(W, g, h)
    R = [[float(W[i, j]) for j in range(N)] for i in range(M)]
    for k in range(K):
        for i in range(M):
            for j in range(N):
                s = -1.0 if R[i][j] < 0 else 1.0
                assert _sign(planes, k, i, j) == s
                R[i][j] -= g[k, i] * s * h[k, j]
    assert _sign(planes, 0, 2, 5) == 1.0


def test_derive_planes_float32_mode_brute_force():
    """The float32 mode (the device kernel's precision) against a scalar loop that rounds to float32 after
    every update; inputs are fp16-valued scales and a float32 weight built so that the two precisions
    disagree somewhere (residuals within float32 rounding of zero)."""
    rng = np.random.default_rng(7)
    K, M, N = 3, 6, 64
    g = (np.abs(rng.standard_normal((K, M))) * np.array([1.0, 0.4, 0.15])[:, None]).astype(np.float16)
    h = rng.uniform(0.5, 1.5, (K, N)).astype(np.float16)
    W = rng.standard_normal((M, N)).astype(np.float32)
    # a row whose first residual is an exact or near tie: W = g_0 * h_0 (+ one float32 ulp on odd columns)
    tie = (g[0, 1].astype(np.float32) * h[0].astype(np.float32)).astype(np.float32)
    W[1] = tie
    W[1, 1::2] = np.nextafter(tie[1::2], np.float32(np.inf))
    planes = orc.derive_planes(W, g, h, dtype=np.float32)
    f32 = np.float32
    for i in range(M):
        for j in range(N):
            r = f32(W[i, j])
            for k in range(K):
                neg = r < 0
                assert _sign(planes, k, i, j) == (-1.0 if neg else 1.0)
                gb = f32(-g[k, i]) if neg else f32(g[k, i])
                r = f32(r - f32(gb * f32(h[k, j])))
    # exact ties give residual +0 -> sign +1 in the next plane
    assert all(_sign(planes, 1, 1, j) == 1.0 for j in range(0, N, 2))
    # and float64 agrees wherever no residual comes within rounding of zero (all rows but the tie row)
    p64 = orc.derive_planes(W.astype(np.float64), g, h)
    keep = [i for i in range(M) if i != 1]
    assert np.array_equal(planes[:, keep], p64[:, keep])


def test_derived_paths_shrink_the_residual():
    """With the mean-magnitude scale each added path lowers ||W - W_hat||_F (error compensation)."""
    rng = np.random.default_rng(6)
    M, N = 64, 128
    W = rng.standard_normal((M, N)) * 0.02
    h = np.ones((2, N))
    g = np.empty((2, M))
    g[0] = np.abs(W).mean(axis=1)
    planes1 = orc.derive_planes(W, g[:1], h[:1])
    R1 = W - orc.dense_weight(planes1, g[:1], h[:1])
    g[1] = np.abs(R1).mean(axis=1)
    planes2 = orc.derive_planes(W, g, h)
    assert np.array_equal(planes2[0], planes1[0])
    R2 = W - orc.dense_weight(planes2, g, h)
    assert np.linalg.norm(R1) < np.linalg.norm(W)
    assert np.linalg.norm(R2) < np.linalg.norm(R1)
    # the second plane is the sign pattern of the first residual
    assert np.array_equal(orc.unpack_signs(planes2, N)[1], np.where(R1 < 0, -1.0, 1.0))


# ---------------------------------------------------------------------------------------
# the generator draws what the recipe says (sanity of the shared inputs, no method arithmetic)
# ---------------------------------------------------------------------------------------
def test_generator_recipe():
    L = make_layer(256, 512, 2, key=(0, 0, 0))
    assert L.planes.dtype == np.uint32 and L.planes.shape == (2, 256, 16)
    assert L.g.dtype == np.float16 and L.h.dtype == np.float16
    h = L.h.astype(np.float64); g = L.g.astype(np.float64)
    assert 0.5 <= h.min() and h.max() <= 1.5
    assert 0.0099 <= g[0].min() and g[0].max() <= 0.0301
    r = g[1] / g[0]
    assert 0.19 <= r.min() and r.max() <= 0.51
    ones = sum(int(w).bit_count() for w in L.planes.ravel())
    assert abs(ones / (2 * 256 * 512) - 0.5) < 0.01
    L2 = make_layer(256, 512, 2, key=(0, 0, 0))
    assert np.array_equal(L.planes, L2.planes) and np.array_equal(L.g, L2.g)
    L3 = make_layer(256, 512, 2, key=(0, 0, 1))
    assert not np.array_equal(L.planes, L3.planes)


def _derive_inputs(K, M, N, seed):
    rng = np.random.default_rng(seed)
    W = (rng.standard_normal((M, N)) * 0.02).astype(np.float32)
    h = rng.uniform(0.5, 1.5, (K, N)).astype(np.float16)
    g = np.empty((K, M), dtype=np.float16)
    scale = 0.016
    for k in range(K):
        g[k] = (scale * rng.uniform(0.8, 1.2, M)).astype(np.float16)
        scale *= 0.45
    return W, g, h


def test_float32_and_float64_readings_differ_only_at_near_ties():
    """Reading R13: the device keeps the residual in fp32.  Against the float64 recurrence of the oracle the planes may
    differ only where a residual is within rounding distance of zero; counted and bounded here."""
    W, g, h = _derive_inputs(3, 512, 1024, seed=5)
    p32 = orc.derive_planes(W, g, h, dtype=np.float32)
    p64 = orc.derive_planes(W, g, h, dtype=np.float64)
    diff = np.unpackbits((p32 ^ p64).view(np.uint8)).sum()
    total = p32.size * 32
    assert np.array_equal(p32[0], p64[0])                                 # the first plane is sign(W) in both
    assert diff / total < 1e-5, f"{diff} of {total} signs differ"
    print(f"fp32 vs float64 derivation: {diff} of {total} signs differ ({diff / total:.2e})")



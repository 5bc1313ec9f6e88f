"""CPU float64 oracle for the residual-binary linear layer.  TEST INFRASTRUCTURE ONLY.

Nothing in the product path may import this module; it exists so that tests, the smoke
check and the benchmark's CPU-baseline leg can compare the CUDA library with a plain,
slow, obviously-correct statement of what the layer computes.  It shares no code with the
CUDA path and is never tuned for speed.

What it computes (all arithmetic in float64; fp16 inputs convert exactly):

* Section 4.1, dual-scale binary block: a path's weight is ``(W_k)_ij = g_k[i] * B_k[i,j] * h_k[j]``
  with ``B_k`` in {-1,+1}, ``g_k`` per output row and ``h_k`` per input column.
* Eq. 2 (stacked binary weight): ``W = sum_k W_k``.
* Section 4.1 forward: ``y = W x``  (equal to ``sum_k g_k * (B_k (h_k * x))``).
* Appendix "Weight Packing": a sign is stored as one bit, +1 -> 0 and -1 -> 1, 32 input
  columns per 32-bit word.  The paper does not fix the bit order inside a word; the reading
  taken here is LSB first (column j -> bit j % 32 of word j // 32).

Pins (tests/test_oracle_pins.py): brute-force triple loop on tiny shapes, the K=1 closed
form, linearity, constant-sign planes, unit-vector probes of single entries, the all-ones
popcount identity, Eq. 2 entry by entry, the storage accounting printed in Section 4.1
(about 2.02 effective bits for a nominal 2-bit layer).  No function here is unpinned.
"""
from __future__ import annotations

import numpy as np


def unpack_signs(planes: np.ndarray, N: int) -> np.ndarray:
    """Sign matrices ``B`` as float64 ``[K][M][N]`` with entries +-1.

    Appendix "Weight Packing": bit 0 is +1 and bit 1 is -1, so ``B = 1 - 2 * bit``; column j
    is bit ``j % 32`` of word ``j // 32`` (LSB-first reading).
    """
    planes = np.asarray(planes, dtype=np.uint32)
    K, M, words = planes.shape
    if words * 32 != N:
        raise ValueError("planes must hold N/32 words per row")
    shifts = np.arange(32, dtype=np.uint32)
    bits = (planes[:, :, :, None] >> shifts) & np.uint32(1)      # [K][M][N/32][32]
    bits = bits.reshape(K, M, N).astype(np.float64)
    return 1.0 - 2.0 * bits


def dense_weight(planes: np.ndarray, g: np.ndarray, h: np.ndarray) -> np.ndarray:
    """Eq. 2: ``W[i,j] = sum_k g_k[i] * B_k[i,j] * h_k[j]`` as a dense float64 ``[M][N]``."""
    g = np.asarray(g, dtype=np.float64)
    h = np.asarray(h, dtype=np.float64)
    K, M = g.shape
    N = h.shape[1]
    B = unpack_signs(planes, N)
    W = np.zeros((M, N), dtype=np.float64)
    for k in range(K):
        W += g[k][:, None] * B[k] * h[k][None, :]
    return W


def linear(planes: np.ndarray, g: np.ndarray, h: np.ndarray, x: np.ndarray,
           row_block: int = 512) -> np.ndarray:
    """Section 4.1 forward with the Eq. 2 weight: ``y[b] = W x[b]``; returns float64 ``[batch][M]``.

    The dense weight is formed ``row_block`` output rows at a time only to bound memory;
    each block is exactly ``dense_weight`` of those rows followed by one float64 product.
    """
    planes = np.asarray(planes, dtype=np.uint32)
    g = np.asarray(g, dtype=np.float64)
    h = np.asarray(h, dtype=np.float64)
    x = np.asarray(x, dtype=np.float64)
    if x.ndim == 1:
        x = x[None, :]
    K, M = g.shape
    y = np.empty((x.shape[0], M), dtype=np.float64)
    for r0 in range(0, M, row_block):
        r1 = min(M, r0 + row_block)
        W = dense_weight(planes[:, r0:r1, :], g[:, r0:r1], h)
        y[:, r0:r1] = x @ W.T
    return y


def l1_bound(g: np.ndarray, h: np.ndarray, x: np.ndarray) -> np.ndarray:
    """``max_i sum_j sum_k |g_k[i] h_k[j] x[b,j]|`` per batch column (float64 ``[batch]``).

    This is the largest row sum of ``|W_k| |x|`` over paths, the magnitude the parity
    tolerance is stated against; the inner sum factorises as ``|g_k[i]| * sum_j |h_k[j] x_j|``.
    """
    g = np.abs(np.asarray(g, dtype=np.float64))
    h = np.abs(np.asarray(h, dtype=np.float64))
    x = np.abs(np.asarray(x, dtype=np.float64))
    if x.ndim == 1:
        x = x[None, :]
    col = x @ h.T                      # [batch][K]: sum_j |h_k[j] x[b,j]|
    per_row = col @ g                  # [batch][M]: sum_k |g_k[i]| * col[b,k]
    return per_row.max(axis=1)


def tolerance(g: np.ndarray, h: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Allowed ``max_i |y_gpu - y_ref|`` per batch column: ``2e-3 * l1_bound + 1e-5``."""
    return 2e-3 * l1_bound(g, h, x) + 1e-5


def storage_bits_per_weight(K: int, M: int, N: int, scale_bits: int = 16) -> float:
    """Section 4.1 storage accounting: K sign bits per weight plus the scale vectors."""
    return (K * M * N + scale_bits * K * (M + N)) / float(M * N)


def derive_planes(W: np.ndarray, g: np.ndarray, h: np.ndarray, dtype=np.float64) -> np.ndarray:
    """Section 4.2 steps 1-3 / Algorithm 2: ``B_i = sign(R_{i-1})``, ``R_i = R_{i-1} - g_i*B_i*h_i``,
    ``R_0 = W``.  Returns canonical packed planes uint32 ``[K][M][N/32]``.

    The paper does not define sign(0); the reading taken here is sign(0) = +1 (bit 0).  Nor does it
    say in which precision the residual is kept.  A sign is an integer decided by floating point, so
    a comparison with the CUDA path must decide it in the same precision: ``dtype=np.float32`` keeps
    ``R`` in float32 and evaluates ``R - (g*B)*h`` with one rounding per update (``g*B`` and the
    product of two float16 values are exact in float32), which is what the device kernel does.
    The default float64 is the reference for everything else.
    """
    W = np.asarray(W, dtype=dtype)
    g = np.asarray(g, dtype=dtype)
    h = np.asarray(h, dtype=dtype)
    K, M = g.shape
    N = h.shape[1]
    R = W.copy()
    planes = np.zeros((K, M, N // 32), dtype=np.uint32)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    one = dtype(1.0)
    for k in range(K):
        neg = R < 0                                            # bit 1 <=> sign -1
        B = np.where(neg, -one, one).astype(dtype)
        words = (neg.reshape(M, N // 32, 32).astype(np.uint64) * weights).sum(axis=2)
        planes[k] = words.astype(np.uint32)
        R = (R - (g[k][:, None] * B) * h[k][None, :]).astype(dtype)
    return planes

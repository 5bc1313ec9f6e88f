"""Seeded generators for residual-binary linear layers and their activations.

Canonical (layout-free) formats produced here and consumed by both the oracle and the
CUDA library:

* ``planes``  uint32 ``[K][M][N/32]`` -- sign bits, 32 consecutive input columns per word,
  column ``j`` lives in bit ``j % 32`` (LSB first) of word ``j // 32``; bit 1 means -1,
  bit 0 means +1 (the packing rule of the paper's Appendix "Weight Packing").
* ``g``       float16 ``[K][M]``  per-output scale of each path (Section 4.1).
* ``h``       float16 ``[K][N]``  per-input scale of each path (Section 4.1).
* ``x``       float16 ``[batch][N]`` activations, row-major.

Value distributions (the recipe of the benchmark configurations): sign words iid uniform
(every sign is +-1 with p = 0.5), ``h ~ U(0.5, 1.5)``, ``g_1 ~ U(0.01, 0.03)``,
``g_k = g_{k-1} * U(0.2, 0.5)`` for k >= 2, ``x ~ N(0, 1)``; each drawn in float64 and
rounded to float16 (round to nearest even).  These stand in for trained Llama-shaped
layers, which are not available offline.

Seeding rule: every array is drawn from ``numpy.random.default_rng(SeedSequence(key))``
where ``key`` is a tuple of non-negative integers chosen by the caller, e.g.
``(config, layer, projection)`` for weights and ``(config, 10_000 + token)`` for
activations, so any single layer or token can be regenerated without the others.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Iterable, List, Sequence, Tuple

import numpy as np


@dataclass(frozen=True)
class LayerShape:
    name: str
    M: int  # d_out
    N: int  # d_in


@dataclass
class LayerInputs:
    K: int
    M: int
    N: int
    planes: np.ndarray  # uint32 [K][M][N/32]
    g: np.ndarray       # float16 [K][M]
    h: np.ndarray       # float16 [K][N]


CONFIG0_SHAPE = LayerShape("square4096", 4096, 4096)


def llama2_7b_layer_shapes() -> List[LayerShape]:
    """The seven projections of one 7B-shaped decoder layer (d=4096, ffn=11008)."""
    d, f = 4096, 11008
    return [
        LayerShape("q", d, d), LayerShape("k", d, d), LayerShape("v", d, d), LayerShape("o", d, d),
        LayerShape("gate", f, d), LayerShape("up", f, d), LayerShape("down", d, f),
    ]


def llama3_8b_layer_shapes() -> List[LayerShape]:
    """8B-shaped projections (d=4096, kv=1024, ffn=14336)."""
    d, kv, f = 4096, 1024, 14336
    return [
        LayerShape("q", d, d), LayerShape("k", kv, d), LayerShape("v", kv, d), LayerShape("o", d, d),
        LayerShape("gate", f, d), LayerShape("up", f, d), LayerShape("down", d, f),
    ]


def llama_70b_layer_shapes() -> List[LayerShape]:
    """70B-shaped projections (d=8192, kv=1024, ffn=28672), one of each distinct shape."""
    d, kv, f = 8192, 1024, 28672
    return [
        LayerShape("q", d, d), LayerShape("k", kv, d), LayerShape("gate", f, d), LayerShape("down", d, f),
    ]


def _rng(key: Sequence[int]) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([int(v) for v in key]))


def make_layer(M: int, N: int, K: int = 2, key: Sequence[int] = (0,)) -> LayerInputs:
    """Draw one layer: iid sign words and the fp16 scale vectors."""
    if N % 32 != 0:
        raise ValueError("N must be a multiple of 32")
    rng = _rng(tuple(key) + (1,))
    planes = rng.integers(0, 1 << 32, size=(K, M, N // 32), dtype=np.uint64).astype(np.uint32)
    h = rng.uniform(0.5, 1.5, size=(K, N)).astype(np.float16)
    g = np.empty((K, M), dtype=np.float16)
    g[0] = rng.uniform(0.01, 0.03, size=M).astype(np.float16)
    for k in range(1, K):
        u = rng.uniform(0.2, 0.5, size=M)
        g[k] = (g[k - 1].astype(np.float64) * u).astype(np.float16)
    return LayerInputs(K=K, M=M, N=N, planes=planes, g=g, h=h)


def make_x(batch: int, N: int, key: Sequence[int] = (0,)) -> np.ndarray:
    """Draw activations ``[batch][N]`` ~ N(0,1), rounded to float16."""
    rng = _rng(tuple(key) + (2,))
    return rng.standard_normal(size=(batch, N)).astype(np.float16)


def make_planes_constant(K: int, M: int, N: int, bit: int) -> np.ndarray:
    """All sign bits equal to ``bit`` (0: every sign +1, 1: every sign -1)."""
    fill = np.uint32(0xFFFFFFFF if bit else 0)
    return np.full((K, M, N // 32), fill, dtype=np.uint32)


def fp16_bits(a: np.ndarray) -> np.ndarray:
    """The raw 16-bit patterns of a float16 array (what crosses the C ABI)."""
    return np.ascontiguousarray(a, dtype=np.float16).view(np.uint16)

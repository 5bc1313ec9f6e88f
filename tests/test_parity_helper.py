"""CPU self-check of the comparison the GPU parity tests use: it must fail when the reference is wrong by one word of
sign bits (four signs, half a look-up byte), also at widths where the mandated tolerance alone would let that through."""
import numpy as np
import pytest

from oracle import rabit_oracle as orc
from synth import make_layer, make_x
from tests.gpu_util import compare, unit_vector_reference


def _as_if_from_the_device(L, x):
    """What an exact kernel returns: the oracle's result rounded once to fp16."""
    return orc.linear(L.planes, L.g, L.h, x).astype(np.float16).astype(np.float64)


@pytest.mark.parametrize("N", [4096, 11008])
def test_one_flipped_word_fails_the_tight_bound(N):
    L = make_layer(64, N, 2, key=(95, N))
    x = make_x(2, N, key=(95, N))
    got = _as_if_from_the_device(L, x)
    l1, tol = orc.l1_bound(L.g, L.h, x), orc.tolerance(L.g, L.h, x)
    compare(got, orc.linear(L.planes, L.g, L.h, x), l1, tol)                 # the true reference passes both bounds
    wrong = L.planes.copy()
    wrong[0, 17, 5] ^= np.uint32(0x00000F00)                                 # four signs of row 17 flipped in the reference copy
    ref_wrong = orc.linear(wrong, L.g, L.h, x)
    assert np.abs(got - ref_wrong).max() <= tol.min()                        # the mandated bound alone would not notice ...
    with pytest.raises(AssertionError, match="tight bound"):
        compare(got, ref_wrong, l1, tol)                                     # ... the tight one does
    compare(got, ref_wrong, l1, tol, tight=False)


def test_unit_vector_reference_is_the_oracle_on_that_input():
    L = make_layer(40, 640, 3, key=(96,))
    for j in (0, 31, 32, 255, 256, 639):
        x = np.zeros((1, 640), dtype=np.float16)
        x[0, j] = 2.5
        assert np.array_equal(unit_vector_reference(L, j, 2.5), orc.linear(L.planes, L.g, L.h, x))

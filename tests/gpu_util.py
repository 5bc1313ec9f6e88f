"""Helpers for the GPU parity tests: run the CUDA library through its C ABI and compare
with the CPU oracle element by element under the stated tolerance."""
import numpy as np

from oracle import rabit_oracle as orc


def run_layer(layer_inputs, x_np, variant=0, device="cuda:0"):
    import torch
    import paper_2602_05367_b200 as rabit

    L = rabit.rabit_pack(layer_inputs.planes, layer_inputs.g, layer_inputs.h, device=device)
    try:
        if variant:
            L.set_variant(variant)
        x = torch.from_numpy(np.ascontiguousarray(x_np)).to(device)
        y = rabit.rabit_linear(L, x)
        torch.cuda.synchronize()
        assert L.status() == 0, rabit.last_error()          # no bounded wait ran out, no index check of a checked build failed
        return y.cpu().numpy()
    finally:
        L.free()


def compare(got, ref, l1, tol, tight=True):
    """The two assertions every parity test makes, per batch row:
      (1) the mandated bound   max_i |y - y_ref| <= 2e-3 * max_i sum_j sum_k |g_ki h_kj x_j| + 1e-5  (= tol)
      (2) a tight bound that the exact-arithmetic kernels also meet,  |y_i - y_ref_i| <= 2^-10 |y_ref_i| + 1e-5 * L1:
          one fp16 rounding of the output plus fp32-level accumulation error.  A dropped or misplaced tile of signs moves
          a row by far more than this even where the mandated bound would still hold (wide layers), so (2) is what
          catches structural mistakes; only the dequantised-tile GEMM (which rounds every weight to fp16) is exempt.
    got, ref: float64 [batch][rows]; l1, tol: [batch]."""
    assert got.shape == ref.shape
    assert np.isfinite(got).all()
    err = np.abs(got - ref)
    worst = int(np.argmax(err.max(axis=1) / tol))
    assert (err.max(axis=1) <= tol).all(), f"batch row {worst}: err {err[worst].max():.3e} > tol {tol[worst]:.3e}"
    if tight:
        bound = 2.0 ** -10 * np.abs(ref) + 1e-5 * l1[:, None]
        bad = err > bound
        if bad.any():
            b, i = np.argwhere(bad)[0]
            raise AssertionError(f"tight bound: batch row {b}, output {i}: |{got[b, i]:.6g} - {ref[b, i]:.6g}| = {err[b, i]:.3e} > {bound[b, i]:.3e} "
                                 f"({int(bad.sum())} outputs off)")
    return err.max(axis=1)


def check_against_oracle(layer_inputs, x_np, y_gpu, tight=True, rows=None):
    """Compare y_gpu [batch][M] (or its columns `rows`) with the oracle on the same inputs."""
    L = layer_inputs
    if rows is None:
        ref = orc.linear(L.planes, L.g, L.h, x_np)
        got = y_gpu.astype(np.float64)
    else:
        ref = orc.linear(L.planes[:, rows, :], L.g[:, rows], L.h, x_np)     # each row of the layer is an independent dot product
        got = y_gpu[:, rows].astype(np.float64)
        assert np.isfinite(y_gpu.astype(np.float64)).all()
    l1 = orc.l1_bound(L.g, L.h, x_np)                                        # the bound is taken over all rows of the layer
    tol = orc.tolerance(L.g, L.h, x_np)
    err = compare(got, ref, l1, tol, tight)
    return err, tol


def unit_vector_reference(layer_inputs, j, value=1.0):
    """Oracle output for x = value * e_j, from the 32-column sub-layer that holds column j (all other columns meet zeros)."""
    L = layer_inputs
    w = j // 32
    x = np.zeros((1, 32), dtype=np.float16)
    x[0, j % 32] = value
    return orc.linear(L.planes[:, :, w:w + 1], L.g, L.h[:, 32 * w:32 * w + 32], x)

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
        return y.cpu().numpy()
    finally:
        L.free()


def check_against_oracle(layer_inputs, x_np, y_gpu):
    """max_i |y_gpu - y_ref| <= 2e-3 * max_i sum_j sum_k |g_ki h_kj x_j| + 1e-5, per batch row."""
    ref = orc.linear(layer_inputs.planes, layer_inputs.g, layer_inputs.h, x_np)
    tol = orc.tolerance(layer_inputs.g, layer_inputs.h, x_np)
    got = y_gpu.astype(np.float64)
    assert got.shape == ref.shape
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max(axis=1)
    worst = int(np.argmax(err / tol))
    assert (err <= tol).all(), f"batch row {worst}: err {err[worst]:.3e} > tol {tol[worst]:.3e}"
    return err, tol

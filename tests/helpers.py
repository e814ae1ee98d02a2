"""Shared helpers of the GPU parity tests: device upload and the comparison bound."""
import numpy as np
import torch

from paper_2202_03293_b200 import inputs

REL_BOUND = 1e-4   # |gpu - oracle| <= REL_BOUND * sum_k |a*b|, per output element


def operand(shape, seed, tensor_id, dist="uniform", dtype="f32"):
    """Returns (device_tensor, oracle_f32_array) holding identical values."""
    payload, vals = inputs.make(shape, seed, tensor_id, dist, dtype)
    if dtype == "bf16":
        dev = torch.from_numpy(payload.view(np.int16).copy()).cuda().view(torch.bfloat16)
    else:
        dev = torch.from_numpy(payload.copy()).cuda()
    return dev, vals


def assert_within_bound(got: torch.Tensor, want: np.ndarray, sum_abs: np.ndarray, what=""):
    g = got.detach().cpu().numpy().astype(np.float64)
    assert g.shape == want.shape, (g.shape, want.shape)
    nonfinite = ~np.isfinite(g)
    if nonfinite.any():
        idx = tuple(int(i) for i in np.argwhere(nonfinite)[0])
        raise AssertionError(f"{what}: {int(nonfinite.sum())} of {g.size} elements are NaN or infinite (an element the kernel "
                             f"never wrote, or a non-finite result); first at {idx}: got {g[idx]!r}, want {want[idx]!r}")
    err = np.abs(g - want)
    bound = REL_BOUND * sum_abs
    bad = ~(err <= bound)        # written so that a NaN anywhere in the comparison fails it
    if bad.any():
        idx = np.unravel_index(np.argmax(np.where(bad, err - bound, -np.inf)), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} elements outside the bound; worst at {idx}: "
                             f"got {g[idx]!r}, want {want[idx]!r}, err {err[idx]:.3e}, bound {bound[idx]:.3e}")
    with np.errstate(divide="ignore", invalid="ignore"):
        ratio = np.where(sum_abs > 0, err / sum_abs, 0.0)
    return float(ratio.max()) if ratio.size else 0.0

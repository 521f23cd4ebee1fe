"""Shared helpers for the GPU parity tests (tensor marshalling and error metrics only)."""
import numpy as np
import torch

from paper_2107_06419_b200 import inputs

# Parity bars: bf16 inputs with fp32 accumulation; fp32 path.
BF16_MAX, BF16_MEAN = 2e-2, 2e-3
F32_MAX = 1e-4
# Beyond the absolute bars: the error relative to the largest reference entry must be small too
# (the absolute bars are of the order of |O| itself at long Nk and would hide a dropped tile).
BF16_REL_MAX = 1e-2


def bf16_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.to(device) if device else t


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def rand_bits(rng, shape, sigma=1.0):
    return inputs.f32_to_bf16_bits((rng.standard_normal(shape) * sigma).astype(np.float32)).reshape(shape)


def check_bf16(got: np.ndarray, ref: np.ndarray, what=""):
    err = np.abs(got - ref)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    mx, mean = float(err.max()), float(err.mean())
    scale = max(float(np.abs(ref).max()), 1e-30)
    assert mx <= BF16_MAX, "%s: max |dO| = %.3e" % (what, mx)
    assert mean <= BF16_MEAN, "%s: mean |dO| = %.3e" % (what, mean)
    assert mx / scale <= BF16_REL_MAX, "%s: max |dO| / max |O| = %.3e" % (what, mx / scale)
    return mx, mean


def check_f32(got: np.ndarray, ref: np.ndarray, what=""):
    err = np.abs(got - ref)
    assert np.all(np.isfinite(got)), what + ": non-finite output"
    mx = float(err.max())
    assert mx <= F32_MAX, "%s: max |dO| = %.3e" % (what, mx)
    return mx

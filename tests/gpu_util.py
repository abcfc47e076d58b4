"""Helpers for the GPU parity tests: device copies and error reporting."""
import numpy as np
import torch

TOL_F32 = 1e-5   # max abs error with fp32 coefficients (images in [0,1], fp32 accumulation)
TOL_F16 = 2e-3   # max abs error with binary16 coefficients


def dev(a: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def host(t: torch.Tensor) -> np.ndarray:
    return t.detach().cpu().numpy()


def tol_for(coef: np.ndarray) -> float:
    return TOL_F16 if coef.dtype == np.float16 else TOL_F32


def max_abs_err(got: np.ndarray, want: np.ndarray) -> float:
    return float(np.max(np.abs(got.astype(np.float64) - want))) if got.size else 0.0

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


def signed_asymmetric_dictionary(dict_: np.ndarray, seed: int = 7) -> np.ndarray:
    """The generator's atoms (point-symmetric, non-negative) made asymmetric and signed.

    Every tap gets N(0, 0.1) noise, and atom 1 becomes a single off-centre delta (tap (0, 1), or the last tap of a
    narrower atom). With such atoms a 180-degree flip of the taps, a transposed patch or a sign slip in the handling
    of negative dictionary values changes the result far beyond the tolerance; with the generator's own atoms
    correlation and convolution agree and none of these would show.
    """
    rng = np.random.default_rng(seed)
    d = dict_.astype(np.float64) + rng.normal(0.0, 0.1, dict_.shape)
    if d.shape[0] > 1 and d.shape[1] > 1:
        d[1] = 0.0
        d[1, 1] = 1.0
    return d.astype(np.float32)


def signed_gamma(s: int, seed: int = 9) -> np.ndarray:
    """Re-weights of a global subset with both signs (every second entry negative) and magnitudes in [0.5, 1.5]."""
    rng = np.random.default_rng(seed)
    g = rng.uniform(0.5, 1.5, size=s)
    g[1::2] *= -1.0
    if s == 1:
        g[0] = -g[0]
    return g.astype(np.float32)

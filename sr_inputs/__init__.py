"""Seeded synthetic inputs shared by the CPU oracle's tests and the CUDA library's tests.

Nothing of the method is computed here: the module fills numpy arrays (LR image,
dictionary, coefficient planes) from a counter-based generator written in C
(`gen.c`, built in-tree with gcc on first use).  Both sides then consume the same
bit patterns, so a tolerance only has to cover the GPU's fp32 arithmetic.

Workload shapes follow the five benchmark configurations: an RGB LR frame with
values uniform in [0,1), a dictionary of D Gaussian / difference-of-Gaussians
atoms of k x k taps (each divided by its own sum), and coefficients
1/D + 0.05 * N(0,1) at HR resolution, one set per frame shared by the channels.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "gen.c")
_LIB = os.path.join(_HERE, "libsrinputs.so")

BASE_SEED = 230308999

_lib = None


def build(force: bool = False) -> str:
    """Compile gen.c into libsrinputs.so next to it (skipped when up to date)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        lib.srg_fill_lr.argtypes = [ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int64]
        lib.srg_fill_lr.restype = None
        lib.srg_fill_coef.argtypes = [ctypes.c_uint64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int64,
                                      ctypes.c_double, ctypes.c_double, ctypes.c_int32]
        lib.srg_fill_coef.restype = None
        lib.srg_round_f16.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64]
        lib.srg_round_f16.restype = None
        lib.srg_make_dictionary.argtypes = [ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32]
        lib.srg_make_dictionary.restype = None
        lib.srg_num_threads.argtypes = []
        lib.srg_num_threads.restype = ctypes.c_int32
        _lib = lib
    return _lib


@dataclass(frozen=True)
class Workload:
    """Shape of one problem: LR batch n x c x h x w, scale r, D atoms of k x k, coefficient dtype."""
    name: str
    n: int
    c: int
    h: int
    w: int
    scale: int
    D: int = 72
    k: int = 5
    coef_dtype: str = "f16"   # "f16" | "f32"
    s: int = 8                # atoms kept per pixel on the selective path

    @property
    def H(self) -> int:
        return self.h * self.scale

    @property
    def W(self) -> int:
        return self.w * self.scale

    @property
    def npix(self) -> int:
        return self.n * self.H * self.W


# The benchmark configurations (cfg4 is a sweep; its anchor point is listed here).
CONFIGS = {
    "cfg0": Workload("cfg0", 1, 3, 64, 64, 2, coef_dtype="f32"),
    "cfg1": Workload("cfg1", 1, 3, 270, 480, 4),
    "cfg2": Workload("cfg2", 1, 3, 270, 480, 4),
    "cfg3": Workload("cfg3", 4, 3, 1080, 1920, 2),
    "cfg4": Workload("cfg4", 1, 3, 360, 640, 3),
}


def cfg4_points():
    """Every point of the shape sweep: scale x D x k on a 360x640 LR frame."""
    for r in (2, 3, 4):
        for D in (16, 32, 72, 128):
            for k in (3, 5, 7):
                yield Workload(f"cfg4_r{r}_D{D}_k{k}", 1, 3, 360, 640, r, D=D, k=k)


def make_lr(wl: Workload, seed: int = BASE_SEED) -> np.ndarray:
    out = np.empty((wl.n, wl.c, wl.h, wl.w), dtype=np.float32)
    _load().srg_fill_lr(seed, out.ctypes.data, out.size)
    return out


def make_dictionary(D: int, k: int, seed: int = BASE_SEED) -> np.ndarray:
    out = np.empty((D, k * k), dtype=np.float32)
    _load().srg_make_dictionary(seed, out.ctypes.data, D, k)
    return out


def make_coef(wl: Workload, seed: int = BASE_SEED, out: np.ndarray | None = None) -> np.ndarray:
    """Coefficients [n][D][H][W]; float16 or float32 according to wl.coef_dtype."""
    dt = np.float16 if wl.coef_dtype == "f16" else np.float32
    if out is None:
        out = np.empty((wl.n, wl.D, wl.H, wl.W), dtype=dt)
    assert out.dtype == dt and out.shape == (wl.n, wl.D, wl.H, wl.W) and out.flags.c_contiguous
    per = wl.D * wl.H * wl.W
    lib = _load()
    for f in range(wl.n):
        lib.srg_fill_coef(seed, f, out[f].ctypes.data, per, 1.0 / wl.D, 0.05, 1 if dt == np.float16 else 0)
    return out


def round_f16(x: np.ndarray) -> np.ndarray:
    """fp32 -> float16 with round-to-nearest-even, through the generator's own routine."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.float16)
    _load().srg_round_f16(x.ctypes.data, out.ctypes.data, x.size)
    return out


def make_inputs(wl: Workload, seed: int = BASE_SEED):
    """Returns (lr, dict, coef) for a workload."""
    return make_lr(wl, seed), make_dictionary(wl.D, wl.k, seed), make_coef(wl, seed)


def num_threads() -> int:
    return int(_load().srg_num_threads())


def make_producer(wl: Workload, cin: int = 32, kc: int = 3, seed: int = BASE_SEED):
    """Inputs of the fused last layer: LR feature map feat [n][h][w][cin] float16 ~ N(0.5, 0.25), the weights of the
    last convolution wconv [D r^2][cin][kc][kc] fp32 ~ N(0, sigma_w) and its bias [D r^2] fp32 ~ 1/D + N(0, 0.005),
    with sigma_w chosen so that the coefficients the layer produces are distributed like the ones make_coef draws
    (mean 1/D, standard deviation 0.05). Stand-ins for a trained network's features and weights."""
    lib = _load()
    r2 = wl.scale * wl.scale
    feat = np.empty((wl.n, wl.h, wl.w, cin), dtype=np.float16)
    lib.srg_fill_coef(seed, 1000, feat.ctypes.data, feat.size, 0.5, 0.25, 1)
    wconv = np.empty((wl.D * r2, cin, kc, kc), dtype=np.float32)
    sigma_w = 0.05 / float(np.sqrt(cin * kc * kc * (0.25 + 0.0625)))
    lib.srg_fill_coef(seed, 1001, wconv.ctypes.data, wconv.size, 0.0, sigma_w, 0)
    bias = np.empty((wl.D * r2,), dtype=np.float32)
    lib.srg_fill_coef(seed, 1002, bias.ctypes.data, bias.size, 1.0 / wl.D, 0.005, 0)
    return feat, wconv, bias

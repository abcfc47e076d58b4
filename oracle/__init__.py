"""ctypes binding of the fp64 CPU oracle (`sr_ref.cpp`).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's cpu_baseline / reference legs.  The CUDA package never imports it.
Arrays are numpy, outputs are float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sr_ref.cpp")
_LIB = os.path.join(_HERE, "libsr_ref.so")

F32, F16 = 0, 1
CLAMP01, IDX_GLOBAL, COEF_COMPACT, UPSAMPLE_BILINEAR, OUT_U8, LUMA_ONLY = 1, 2, 4, 8, 32, 64

_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with g++ -O2 (plus OpenMP for the row loop) into libsr_ref.so."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        vp, i32, i64, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_uint
        L.sr_ref_bicubic_upsample.argtypes = [vp, vp] + [i32] * 6
        L.sr_ref_bilinear_upsample.argtypes = [vp, vp] + [i32] * 6
        L.sr_ref_dict_regress_dense.argtypes = [vp, vp, i32, vp, vp] + [i32] * 7 + [u32, i32]
        L.sr_ref_dict_select.argtypes = [vp, i32, vp, vp] + [i32] * 6
        L.sr_ref_dict_regress_selected.argtypes = [vp, vp, i32, vp, vp, vp, vp] + [i32] * 8 + [u32, i32]
        L.sr_ref_regress_at.argtypes = [i32, vp, vp, i32, vp, vp, vp, vp, i64, vp] + [i32] * 8 + [u32, i32]
        L.sr_ref_dict_select_at.argtypes = [vp, i32, vp, i64, vp] + [i32] * 6
        f64 = ctypes.c_double
        L.sr_ref_selection_gram.argtypes = [vp, vp, i32, vp, vp, vp, i64, vp, vp, vp] + [i32] * 7 + [u32, i32]
        L.sr_ref_lasso_cd.argtypes = [vp, vp, i32, vp, f64, f64, vp, f64, i32, vp]
        L.sr_ref_selection_search.argtypes = [vp, vp, f64, i32, f64, f64, f64, f64, f64, f64, i32, i32, vp, vp, vp, vp, i32, vp]
        for f in (L.sr_ref_selection_gram, L.sr_ref_lasso_cd, L.sr_ref_selection_search):
            f.restype = i32
        L.sr_ref_producer_coef.argtypes = [vp, vp, vp, vp] + [i32] * 8
        L.sr_ref_producer_regress.argtypes = [vp, vp, vp, vp, vp, vp, vp, i32, vp] + [i32] * 9 + [u32, i32]
        L.sr_ref_max_threads.argtypes = []
        for f in (L.sr_ref_bicubic_upsample, L.sr_ref_bilinear_upsample, L.sr_ref_dict_regress_dense, L.sr_ref_dict_select,
                  L.sr_ref_dict_regress_selected, L.sr_ref_regress_at, L.sr_ref_dict_select_at, L.sr_ref_max_threads):
            f.restype = i32
        _lib = L
    return _lib


def max_threads() -> int:
    return int(_load().sr_ref_max_threads())


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.float16:
        return F16
    raise TypeError(f"coefficients must be float32 or float16, got {a.dtype}")


def _c(a, dt=None):
    a = np.ascontiguousarray(a) if dt is None else np.ascontiguousarray(a, dtype=dt)
    return a


def _check(status: int, what: str):
    if status != 0:
        raise ValueError(f"{what}: oracle status {status}")


def bicubic_upsample(lr: np.ndarray, scale: int, threads: int = 0) -> np.ndarray:
    lr = _c(lr, np.float32)
    n, c, h, w = lr.shape
    out = np.empty((n, c, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_bicubic_upsample(lr.ctypes.data, out.ctypes.data, n, c, h, w, scale, threads), "bicubic")
    return out


def bilinear_upsample(lr: np.ndarray, scale: int, threads: int = 0) -> np.ndarray:
    lr = _c(lr, np.float32)
    n, c, h, w = lr.shape
    out = np.empty((n, c, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_bilinear_upsample(lr.ctypes.data, out.ctypes.data, n, c, h, w, scale, threads), "bilinear")
    return out


def dict_regress_dense(lr, coef, dict_, scale: int, k: int, flags: int = 0, threads: int = 0) -> np.ndarray:
    lr, coef, dict_ = _c(lr, np.float32), _c(coef), _c(dict_, np.float32)
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    assert dict_.shape == (D, k * k) and coef.shape == (n, D, h * scale, w * scale), (dict_.shape, coef.shape)
    out = np.empty((n, c, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_dict_regress_dense(lr.ctypes.data, coef.ctypes.data, _dtype_code(coef), dict_.ctypes.data,
                                             out.ctypes.data, n, c, h, w, scale, k, D, flags, threads), "dense")
    return out


def dict_select(coef, s: int, want_sel: bool = False, threads: int = 0):
    coef = _c(coef)
    n, D, H, W = coef.shape
    idx = np.empty((n, s, H, W), dtype=np.uint8)
    sel = np.empty((n, s, H, W), dtype=np.float64) if want_sel else None
    _check(_load().sr_ref_dict_select(coef.ctypes.data, _dtype_code(coef), idx.ctypes.data,
                                      sel.ctypes.data if want_sel else None, n, H, W, D, s, threads), "select")
    return (idx, sel) if want_sel else idx


def dict_regress_selected(lr, coef_or_sel, idx, gamma, dict_, scale: int, k: int, s: int, flags: int = 0,
                          threads: int = 0) -> np.ndarray:
    lr, coef_or_sel, dict_ = _c(lr, np.float32), _c(coef_or_sel), _c(dict_, np.float32)
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    idx = None if idx is None else _c(idx, np.uint8)
    gamma = None if gamma is None else _c(gamma, np.float32)
    out = np.empty((n, c, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_dict_regress_selected(
        lr.ctypes.data, coef_or_sel.ctypes.data, _dtype_code(coef_or_sel), None if idx is None else idx.ctypes.data,
        None if gamma is None else gamma.ctypes.data, dict_.ctypes.data, out.ctypes.data, n, c, h, w, scale, k, D, s,
        flags, threads), "selected")
    return out


def regress_at(mode: str, lr, coef_or_sel, idx, gamma, dict_, samples, scale: int, k: int, s: int = 0, flags: int = 0,
               threads: int = 0) -> np.ndarray:
    """Dense (`mode="dense"`) or selected regression at sampled flat [n][H][W] indices -> [nsamples][c]."""
    lr, coef_or_sel, dict_ = _c(lr, np.float32), _c(coef_or_sel), _c(dict_, np.float32)
    samples = _c(samples, np.int64)
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    idx = None if idx is None else _c(idx, np.uint8)
    gamma = None if gamma is None else _c(gamma, np.float32)
    out = np.empty((samples.size, c), dtype=np.float64)
    _check(_load().sr_ref_regress_at(
        0 if mode == "dense" else 1, lr.ctypes.data, coef_or_sel.ctypes.data, _dtype_code(coef_or_sel),
        None if idx is None else idx.ctypes.data, None if gamma is None else gamma.ctypes.data, dict_.ctypes.data,
        samples.ctypes.data, samples.size, out.ctypes.data, n, c, h, w, scale, k, D, s if s else D, flags, threads),
        "regress_at")
    return out


def dict_select_at(coef, samples, s: int, threads: int = 0) -> np.ndarray:
    coef = _c(coef)
    samples = _c(samples, np.int64)
    n, D, H, W = coef.shape
    out = np.empty((samples.size, s), dtype=np.uint8)
    _check(_load().sr_ref_dict_select_at(coef.ctypes.data, _dtype_code(coef), samples.ctypes.data, samples.size,
                                         out.ctypes.data, n, H, W, D, s, threads), "select_at")
    return out


def selection_gram(lr, coef, dict_, target, samples, scale: int, k: int, flags: int = 0, threads: int = 0):
    """Gram statistics of the selection problem (Section III-A) over sampled flat [n][H][W] pixel indices
    (None = every pixel): returns (G [L][L], b [L], hh) in float64."""
    lr, coef, dict_, target = _c(lr, np.float32), _c(coef), _c(dict_, np.float32), _c(target, np.float32)
    n, c, h, w = lr.shape
    L = dict_.shape[0]
    assert dict_.shape == (L, k * k) and coef.shape == (n, L, h * scale, w * scale) and target.shape == (n, c, h * scale, w * scale)
    samples = None if samples is None else _c(samples, np.int64)
    G = np.empty((L, L), dtype=np.float64)
    b = np.empty(L, dtype=np.float64)
    hh = ctypes.c_double(0.0)
    _check(_load().sr_ref_selection_gram(lr.ctypes.data, coef.ctypes.data, _dtype_code(coef), dict_.ctypes.data, target.ctypes.data,
                                         None if samples is None else samples.ctypes.data, 0 if samples is None else samples.size,
                                         G.ctypes.data, b.ctypes.data, ctypes.addressof(hh), n, c, h, w, scale, k, L, flags, threads),
           "selection_gram")
    return G, b, float(hh.value)


def lasso_cd(G, b, nrows: float, lam: float, beta0=None, active=None, tol: float = 1e-12, max_sweeps: int = 10000):
    """Eq. 7 for one lambda by cyclic coordinate descent on the Gram matrix: returns (beta, sweeps)."""
    G, b = _c(G, np.float64), _c(b, np.float64)
    L = b.size
    beta = np.ones(L) if beta0 is None else np.array(beta0, dtype=np.float64)
    act = np.ones(L, dtype=np.uint8) if active is None else _c(active, np.uint8)
    sweeps = ctypes.c_int(0)
    _check(_load().sr_ref_lasso_cd(G.ctypes.data, b.ctypes.data, L, act.ctypes.data, float(nrows), float(lam), beta.ctypes.data,
                                   float(tol), int(max_sweeps), ctypes.addressof(sweeps)), "lasso_cd")
    return beta, int(sweeps.value)


def selection_search(G, b, hh: float, nrows: float, alpha: float, delta_alpha: float, eps: float, lambda0: float,
                     tol: float = 1e-12, max_sweeps: int = 10000, max_bisect: int = 30, max_steps: int = 64):
    """Algorithm 1 on the Gram statistics: returns (idx uint8 [count], gamma float64 [count], trace [steps][6])."""
    G, b = _c(G, np.float64), _c(b, np.float64)
    L = b.size
    idx = np.zeros(L, dtype=np.uint8)
    gamma = np.zeros(L, dtype=np.float64)
    trace = np.zeros((max_steps, 6), dtype=np.float64)
    count, steps = ctypes.c_int(0), ctypes.c_int(0)
    _check(_load().sr_ref_selection_search(G.ctypes.data, b.ctypes.data, float(hh), L, float(nrows), float(alpha), float(delta_alpha),
                                           float(eps), float(lambda0), float(tol), int(max_sweeps), int(max_bisect), idx.ctypes.data,
                                           gamma.ctypes.data, ctypes.addressof(count), trace.ctypes.data, max_steps,
                                           ctypes.addressof(steps)), "selection_search")
    return idx[: count.value].copy(), gamma[: count.value].copy(), trace[: steps.value].copy()


def producer_coef(feat, wconv, bias, scale: int, threads: int = 0) -> np.ndarray:
    """Phi [n][L][H][W] (fp64) from the LR feature map feat [n][h][w][cin] (float16), the last convolution
    wconv [L r^2][cin][kc][kc] (+ bias [L r^2] or None) and the pixel-shuffle by `scale`."""
    feat, wconv = _c(feat, np.float16), _c(wconv, np.float32)
    n, h, w, cin = feat.shape
    cout, cin2, kc, kc2 = wconv.shape
    assert cin2 == cin and kc2 == kc and cout % (scale * scale) == 0
    L = cout // (scale * scale)
    bias = None if bias is None else _c(bias, np.float32)
    assert bias is None or bias.shape == (cout,)
    phi = np.empty((n, L, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_producer_coef(feat.ctypes.data, wconv.ctypes.data, None if bias is None else bias.ctypes.data,
                                        phi.ctypes.data, n, h, w, scale, L, cin, kc, threads), "producer_coef")
    return phi


def producer_regress(lr, feat, wconv, bias, dict_, scale: int, k: int, idx=None, gamma=None, flags: int = 0,
                     threads: int = 0) -> np.ndarray:
    """The dense regression (or the global-subset one, with idx / gamma) with Phi computed from the feature map."""
    lr, feat, wconv, dict_ = _c(lr, np.float32), _c(feat, np.float16), _c(wconv, np.float32), _c(dict_, np.float32)
    n, c, h, w = lr.shape
    assert feat.shape[:3] == (n, h, w)
    cin = feat.shape[3]
    cout, cin2, kc, kc2 = wconv.shape
    D = dict_.shape[0]
    assert cin2 == cin and kc2 == kc and cout == D * scale * scale and dict_.shape == (D, k * k)
    bias = None if bias is None else _c(bias, np.float32)
    idx = None if idx is None else _c(idx, np.uint8)
    gamma = None if gamma is None else _c(gamma, np.float32)
    s = 0 if idx is None else idx.size
    out = np.empty((n, c, h * scale, w * scale), dtype=np.float64)
    _check(_load().sr_ref_producer_regress(
        lr.ctypes.data, feat.ctypes.data, wconv.ctypes.data, None if bias is None else bias.ctypes.data, dict_.ctypes.data,
        None if idx is None else idx.ctypes.data, None if gamma is None else gamma.ctypes.data, s, out.ctypes.data,
        n, c, h, w, scale, k, D, cin, kc, flags, threads), "producer_regress")
    return out

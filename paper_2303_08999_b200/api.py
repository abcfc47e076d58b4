"""Thin Python binding of the C-ABI library (argument marshalling only).

Every function takes torch CUDA tensors (used purely as device memory), checks their dtype, shape and
contiguity, and passes raw pointers, the problem dimensions and the current CUDA stream to the
library entry point of the same name. Nothing is computed in Python and nothing falls back to the CPU:
if the library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsr.so")

SR_F32, SR_F16 = 0, 1
SR_CLAMP01, SR_IDX_GLOBAL, SR_COEF_COMPACT, SR_UPSAMPLE_BILINEAR, SR_OUT_F16, SR_OUT_U8, SR_LUMA_ONLY = 1, 2, 4, 8, 16, 32, 64
SR_OK, SR_ERR_NULL, SR_ERR_SHAPE, SR_ERR_UNSUPPORTED, SR_ERR_ALIGN, SR_ERR_CUDA, SR_ERR_TIMEOUT, SR_ERR_TOO_LARGE = range(8)

EXPORTS = ("sr_bicubic_upsample", "sr_bilinear_upsample", "sr_dict_regress_dense", "sr_dict_select", "sr_dict_regress_selected",
           "sr_status_string", "sr_device_status", "sr_launch_count", "sr_set_wait_limit", "sr_test_lose_arrival", "sr_test_force_kernel",
           "sr_selection_gram", "sr_selection_gram_scratch_bytes", "sr_selection_search", "sr_selection_search_scratch_bytes",
           "sr_selection_gram_static", "sr_probe_rate", "sr_tune_dense", "sr_tune_selected", "sr_tune_reset",
           "sr_producer_folded_bytes", "sr_producer_fold", "sr_producer_regress")


class sr_dims(ctypes.Structure):
    _fields_ = [(name, ctypes.c_int32) for name in ("n", "c", "h", "w", "scale", "k", "D")]


class sr_search_opts(ctypes.Structure):
    _fields_ = [("alpha", ctypes.c_double), ("delta_alpha", ctypes.c_double), ("eps", ctypes.c_double), ("lambda0", ctypes.c_double),
                ("tol", ctypes.c_double), ("max_sweeps", ctypes.c_int32), ("max_bisect", ctypes.c_int32), ("max_steps", ctypes.c_int32)]


class sr_tune_result(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_int32), ("tile_rows", ctypes.c_int32), ("rows_per_step", ctypes.c_int32),
                ("candidates", ctypes.c_int32), ("best_us", ctypes.c_float), ("default_us", ctypes.c_float)]


class SrError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


_lib = None


def load_library() -> ctypes.CDLL:
    """Loads libsr.so; raises if it has not been built (there is no other implementation to fall back to)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2303_08999_b200.build`")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32
        dp = ctypes.POINTER(sr_dims)
        lib.sr_bicubic_upsample.argtypes = [vp, vp, dp, vp]
        lib.sr_bilinear_upsample.argtypes = [vp, vp, dp, vp]
        lib.sr_dict_regress_dense.argtypes = [vp, vp, i32, vp, vp, dp, u32, vp]
        lib.sr_dict_select.argtypes = [vp, i32, vp, vp, dp, i32, u32, vp]
        lib.sr_dict_regress_selected.argtypes = [vp, vp, i32, vp, vp, vp, vp, dp, i32, u32, vp]
        lib.sr_device_status.argtypes = [vp, ctypes.POINTER(ctypes.c_int)]
        for name in EXPORTS:
            getattr(lib, name).restype = i32
        lib.sr_tune_reset.restype = None
        lib.sr_launch_count.argtypes = []
        lib.sr_launch_count.restype = ctypes.c_int64
        lib.sr_set_wait_limit.argtypes = [ctypes.c_int64]
        lib.sr_set_wait_limit.restype = ctypes.c_int64
        lib.sr_test_lose_arrival.argtypes = [i32]
        lib.sr_test_force_kernel.argtypes = [i32]
        i64, f64, sz = ctypes.c_int64, ctypes.c_double, ctypes.c_size_t
        lib.sr_selection_gram_scratch_bytes.argtypes = [dp]
        lib.sr_selection_gram_scratch_bytes.restype = sz
        lib.sr_selection_gram.argtypes = [vp, vp, i32, vp, vp, vp, i64, vp, vp, vp, dp, u32, vp, sz, vp]
        tp = ctypes.POINTER(sr_tune_result)
        lib.sr_tune_dense.argtypes = [vp, vp, i32, vp, vp, dp, u32, i32, vp, tp]
        lib.sr_tune_selected.argtypes = [vp, vp, i32, vp, vp, vp, vp, dp, i32, u32, i32, vp, tp]
        lib.sr_tune_reset.argtypes = []
        lib.sr_probe_rate.argtypes = [i32, vp, ctypes.POINTER(ctypes.c_double), vp]
        lib.sr_selection_gram_static.argtypes = [vp, vp, i32, vp, vp, vp, i64, vp, vp, vp, dp, u32, vp]
        lib.sr_selection_search_scratch_bytes.argtypes = [ctypes.c_int32]
        lib.sr_selection_search_scratch_bytes.restype = sz
        lib.sr_selection_search.argtypes = [vp, vp, vp, f64, ctypes.c_int32, ctypes.POINTER(sr_search_opts), vp, vp, vp, vp, vp, vp, sz, vp]
        lib.sr_producer_folded_bytes.argtypes = [dp, i32, i32]
        lib.sr_producer_folded_bytes.restype = sz
        lib.sr_producer_fold.argtypes = [vp, vp, vp, vp, vp, i32, vp, sz, dp, i32, i32, vp]
        lib.sr_producer_regress.argtypes = [vp, vp, vp, sz, vp, dp, i32, i32, u32, vp]
        lib.sr_status_string.argtypes = [i32]
        lib.sr_status_string.restype = ctypes.c_char_p
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load_library().sr_status_string(status).decode()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t):
    return None if t is None else t.data_ptr()


def _dev(t: torch.Tensor, dtype, what: str) -> torch.Tensor:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError(f"{what} must be a contiguous CUDA tensor of {dtype}")
    return t


def _coef_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return SR_F16
    if t.dtype == torch.float32:
        return SR_F32
    raise TypeError("coefficients must be float16 or float32")


def _out_dtype(flags: int):
    return torch.uint8 if (flags & SR_OUT_U8) else (torch.float16 if (flags & SR_OUT_F16) else torch.float32)


def _check(status: int, what: str):
    if status != SR_OK:
        raise SrError(status, what)


def _upsample(name: str, lr: torch.Tensor, scale: int, out: torch.Tensor | None) -> torch.Tensor:
    lr = _dev(lr, torch.float32, "lr")
    n, c, h, w = lr.shape
    if out is None:
        out = torch.empty((n, c, h * scale, w * scale), dtype=torch.float32, device=lr.device)
    _dev(out, torch.float32, "out")
    assert out.shape == (n, c, h * scale, w * scale)
    d = sr_dims(n, c, h, w, scale, 1, 1)
    _check(getattr(load_library(), name)(_ptr(lr), _ptr(out), ctypes.byref(d), _stream()), name)
    return out


def sr_bicubic_upsample(lr: torch.Tensor, scale: int, out: torch.Tensor | None = None) -> torch.Tensor:
    return _upsample("sr_bicubic_upsample", lr, scale, out)


def sr_bilinear_upsample(lr: torch.Tensor, scale: int, out: torch.Tensor | None = None) -> torch.Tensor:
    return _upsample("sr_bilinear_upsample", lr, scale, out)


def sr_dict_regress_dense(lr, coef, dict_, scale: int, k: int, flags: int = 0, out=None) -> torch.Tensor:
    lr, dict_ = _dev(lr, torch.float32, "lr"), _dev(dict_, torch.float32, "dict")
    code = _coef_code(coef)
    _dev(coef, coef.dtype, "coef")
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    assert dict_.shape == (D, k * k) and coef.shape == (n, D, h * scale, w * scale)
    out_dtype = _out_dtype(flags)
    if out is None:
        out = torch.empty((n, c, h * scale, w * scale), dtype=out_dtype, device=lr.device)
    _dev(out, out_dtype, "out")
    assert out.shape == (n, c, h * scale, w * scale)
    d = sr_dims(n, c, h, w, scale, k, D)
    _check(load_library().sr_dict_regress_dense(_ptr(lr), _ptr(coef), code, _ptr(dict_), _ptr(out), ctypes.byref(d),
                                                flags, _stream()), "sr_dict_regress_dense")
    return out


def sr_dict_select(coef, s: int, want_sel: bool = False, idx=None, sel=None):
    code = _coef_code(coef)
    _dev(coef, coef.dtype, "coef")
    n, D, H, W = coef.shape
    if idx is None:
        idx = torch.empty((n, s, H, W), dtype=torch.uint8, device=coef.device)
    _dev(idx, torch.uint8, "idx")
    if want_sel and sel is None:
        sel = torch.empty((n, s, H, W), dtype=coef.dtype, device=coef.device)
    if sel is not None:
        _dev(sel, coef.dtype, "sel")
    d = sr_dims(n, 1, H, W, 1, 1, D)
    _check(load_library().sr_dict_select(_ptr(coef), code, _ptr(idx), _ptr(sel), ctypes.byref(d), s, 0, _stream()),
           "sr_dict_select")
    return (idx, sel) if sel is not None else idx


def sr_dict_regress_selected(lr, coef_or_sel, idx, gamma, dict_, scale: int, k: int, s: int, flags: int = 0,
                             out=None) -> torch.Tensor:
    lr, dict_ = _dev(lr, torch.float32, "lr"), _dev(dict_, torch.float32, "dict")
    code = _coef_code(coef_or_sel)
    _dev(coef_or_sel, coef_or_sel.dtype, "coef_or_sel")
    if idx is not None:
        _dev(idx, torch.uint8, "idx")
    if gamma is not None:
        _dev(gamma, torch.float32, "gamma")
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    assert dict_.shape == (D, k * k)
    planes = s if (flags & SR_COEF_COMPACT) else D
    assert coef_or_sel.shape == (n, planes, h * scale, w * scale)
    out_dtype = _out_dtype(flags)
    if out is None:
        out = torch.empty((n, c, h * scale, w * scale), dtype=out_dtype, device=lr.device)
    _dev(out, out_dtype, "out")
    assert out.shape == (n, c, h * scale, w * scale)
    d = sr_dims(n, c, h, w, scale, k, D)
    _check(load_library().sr_dict_regress_selected(_ptr(lr), _ptr(coef_or_sel), code, _ptr(idx), _ptr(gamma),
                                                   _ptr(dict_), _ptr(out), ctypes.byref(d), s, flags, _stream()),
           "sr_dict_regress_selected")
    return out


def sr_device_status() -> int:
    """Synchronises the current stream and returns (and clears) the device status word."""
    v = ctypes.c_int(0)
    _check(load_library().sr_device_status(_stream(), ctypes.byref(v)), "sr_device_status")
    return v.value


def sr_launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(load_library().sr_launch_count())


def sr_set_wait_limit(cycles: int) -> int:
    """Cycle budget of the device-side waits of later launches; returns the previous budget."""
    return int(load_library().sr_set_wait_limit(int(cycles)))


def sr_test_lose_arrival(launches: int) -> None:
    """Test hook: the next `launches` tensor-core regression launches leave out one barrier arrival."""
    _check(load_library().sr_test_lose_arrival(int(launches)), "sr_test_lose_arrival")


KERNEL_NAMES = {0: "general", 1: "first tensor-core layout", 2: "second tensor-core layout", 3: "subset (FMA pipe)",
                4: "gather (FMA pipe)"}


def sr_test_force_kernel(kernel: int) -> None:
    """Test hook: later regression calls run on kernel `kernel` (a key of KERNEL_NAMES) where it supports them; -1 = host rules."""
    _check(load_library().sr_test_force_kernel(int(kernel)), "sr_test_force_kernel")


def sr_selection_gram(lr, coef, dict_, target, samples, scale: int, k: int, flags: int = 0):
    """Gram statistics of the dictionary selection search: returns (G [D][D], b [D], hh [1]) as float64 CUDA tensors.
    `samples`: int64 CUDA tensor of flat [n][H][W] pixel indices, or None for every pixel."""
    lr, dict_, target = _dev(lr, torch.float32, "lr"), _dev(dict_, torch.float32, "dict"), _dev(target, torch.float32, "target")
    code = _coef_code(coef)
    _dev(coef, coef.dtype, "coef")
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    assert dict_.shape == (D, k * k) and coef.shape == (n, D, h * scale, w * scale) and target.shape == (n, c, h * scale, w * scale)
    if samples is not None:
        _dev(samples, torch.int64, "samples")
    d = sr_dims(n, c, h, w, scale, k, D)
    lib = load_library()
    nbytes = int(lib.sr_selection_gram_scratch_bytes(ctypes.byref(d)))
    if nbytes == 0:
        raise SrError(SR_ERR_UNSUPPORTED, "sr_selection_gram_scratch_bytes")
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=lr.device)
    G = torch.empty((D, D), dtype=torch.float64, device=lr.device)
    b = torch.empty(D, dtype=torch.float64, device=lr.device)
    hh = torch.empty(1, dtype=torch.float64, device=lr.device)
    _check(lib.sr_selection_gram(_ptr(lr), _ptr(coef), code, _ptr(dict_), _ptr(target), _ptr(samples),
                                 0 if samples is None else samples.numel(), _ptr(G), _ptr(b), _ptr(hh), ctypes.byref(d), flags,
                                 _ptr(scratch), nbytes, _stream()), "sr_selection_gram")
    return G, b, hh


def sr_selection_search(G, b, hh, nrows: float, alpha: float, delta_alpha: float, eps: float, lambda0: float, tol: float = 1e-9,
                        max_sweeps: int = 2000, max_bisect: int = 30, max_steps: int = 64):
    """Algorithm 1 on the Gram statistics (float64 CUDA tensors). Returns (idx uint8 [count], gamma float32 [count],
    trace float64 [steps][6]) as CUDA tensors; reading the count synchronises the stream."""
    _dev(G, torch.float64, "G"), _dev(b, torch.float64, "b"), _dev(hh, torch.float64, "hh")
    D = b.numel()
    assert G.shape == (D, D) and hh.numel() == 1
    lib = load_library()
    nbytes = int(lib.sr_selection_search_scratch_bytes(D))
    if nbytes == 0:
        raise SrError(SR_ERR_UNSUPPORTED, "sr_selection_search_scratch_bytes")
    scratch = torch.empty(nbytes, dtype=torch.uint8, device=G.device)
    idx = torch.zeros(D, dtype=torch.uint8, device=G.device)
    gamma = torch.zeros(D, dtype=torch.float32, device=G.device)
    count = torch.zeros(1, dtype=torch.int32, device=G.device)
    steps = torch.zeros(1, dtype=torch.int32, device=G.device)
    trace = torch.zeros((max_steps, 6), dtype=torch.float64, device=G.device)
    o = sr_search_opts(alpha, delta_alpha, eps, lambda0, tol, max_sweeps, max_bisect, max_steps)
    _check(lib.sr_selection_search(_ptr(G), _ptr(b), _ptr(hh), float(nrows), D, ctypes.byref(o), _ptr(idx), _ptr(gamma), _ptr(count),
                                   _ptr(trace), _ptr(steps), _ptr(scratch), nbytes, _stream()), "sr_selection_search")
    n = int(count.item())
    if n < 0:
        raise SrError(SR_ERR_UNSUPPORTED, "sr_selection_search: a re-fit met a singular matrix")
    return idx[:n], gamma[:n], trace[: int(steps.item())]


def sr_probe_rate(kind: int) -> float:
    """Sustained lane operations per second of integer max/min (kind 0), fp32 multiply-add (kind 1) or packed fp32
    multiply-add (kind 2, two per lane and instruction) on the current device."""
    scratch = torch.zeros(2, dtype=torch.int32, device="cuda")
    v = ctypes.c_double(0.0)
    _check(load_library().sr_probe_rate(kind, _ptr(scratch), ctypes.byref(v), _stream()), "sr_probe_rate")
    return float(v.value)


def sr_producer_fold(wconv, bias, dict_, scale: int, k: int, idx=None, gamma=None) -> torch.Tensor:
    """Folds the dictionary (every atom, or the subset idx with weights gamma) into the last convolution's weights
    wconv [D*scale^2][cin][kc][kc] and bias; returns the folded block sr_producer_regress takes."""
    wconv, dict_ = _dev(wconv, torch.float32, "wconv"), _dev(dict_, torch.float32, "dict")
    bias = None if bias is None else _dev(bias, torch.float32, "bias")
    idx = None if idx is None else _dev(idx, torch.uint8, "idx")
    gamma = None if gamma is None else _dev(gamma, torch.float32, "gamma")
    cout, cin, kc, kc2 = wconv.shape
    D = dict_.shape[0]
    if kc2 != kc or cout != D * scale * scale or dict_.shape[1] != k * k or (bias is not None and bias.numel() != cout):
        raise ValueError("shapes of wconv / bias / dict do not agree")
    d = sr_dims(1, 1, 1, 1, scale, k, D)
    lib = load_library()
    nbytes = int(lib.sr_producer_folded_bytes(ctypes.byref(d), cin, kc))
    if nbytes == 0:
        raise SrError(SR_ERR_UNSUPPORTED, "sr_producer_folded_bytes")
    folded = torch.empty(nbytes, dtype=torch.uint8, device=wconv.device)
    _check(lib.sr_producer_fold(_ptr(wconv), _ptr(bias), _ptr(dict_), _ptr(idx), _ptr(gamma), 0 if idx is None else idx.numel(),
                                _ptr(folded), nbytes, ctypes.byref(d), cin, kc, _stream()), "sr_producer_fold")
    return folded


def sr_producer_regress(lr, feat, folded, scale: int, k: int, D: int, kc: int, flags: int = 0, out=None) -> torch.Tensor:
    """Dense (or folded-subset) regression with the coefficients computed on the fly from the LR feature map
    feat [n][h][w][cin] (float16, channels last) and the folded weights."""
    lr, feat = _dev(lr, torch.float32, "lr"), _dev(feat, torch.float16, "feat")
    folded = _dev(folded, torch.uint8, "folded")
    n, c, h, w = lr.shape
    if tuple(feat.shape[:3]) != (n, h, w):
        raise ValueError("feat must be [n][h][w][cin]")
    cin = feat.shape[3]
    if out is None:
        out = torch.empty((n, c, h * scale, w * scale), dtype=_out_dtype(flags), device=lr.device)
    d = sr_dims(n, c, h, w, scale, k, D)
    _check(load_library().sr_producer_regress(_ptr(lr), _ptr(feat), _ptr(folded), folded.numel(), _ptr(out), ctypes.byref(d), cin, kc,
                                              flags, _stream()), "sr_producer_regress")
    return out


def _tune_dict(res: sr_tune_result) -> dict:
    return {"kernel": KERNEL_NAMES.get(res.kernel, str(res.kernel)), "tile_rows": res.tile_rows, "rows_per_step": res.rows_per_step,
            "candidates": res.candidates, "best_us": res.best_us, "default_us": res.default_us}


def sr_tune_dense(lr, coef, dict_, scale: int, k: int, flags: int = 0, reps: int = 5) -> dict:
    """Tile-shape search for sr_dict_regress_dense on these buffers; later calls with the same shape use the result."""
    lr, dict_ = _dev(lr, torch.float32, "lr"), _dev(dict_, torch.float32, "dict")
    code = _coef_code(coef)
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    out = torch.empty((n, c, h * scale, w * scale), dtype=_out_dtype(flags), device=lr.device)
    d = sr_dims(n, c, h, w, scale, k, D)
    res = sr_tune_result()
    _check(load_library().sr_tune_dense(_ptr(lr), _ptr(coef), code, _ptr(dict_), _ptr(out), ctypes.byref(d), flags, reps, _stream(),
                                        ctypes.byref(res)), "sr_tune_dense")
    return _tune_dict(res)


def sr_tune_selected(lr, coef_or_sel, idx, gamma, dict_, scale: int, k: int, s: int, flags: int = 0, reps: int = 5) -> dict:
    """Tile-shape search for sr_dict_regress_selected on these buffers."""
    lr, dict_ = _dev(lr, torch.float32, "lr"), _dev(dict_, torch.float32, "dict")
    code = _coef_code(coef_or_sel)
    n, c, h, w = lr.shape
    D = dict_.shape[0]
    out = torch.empty((n, c, h * scale, w * scale), dtype=_out_dtype(flags), device=lr.device)
    d = sr_dims(n, c, h, w, scale, k, D)
    res = sr_tune_result()
    _check(load_library().sr_tune_selected(_ptr(lr), _ptr(coef_or_sel), code, _ptr(idx), _ptr(gamma), _ptr(dict_), _ptr(out),
                                           ctypes.byref(d), s, flags, reps, _stream(), ctypes.byref(res)), "sr_tune_selected")
    return _tune_dict(res)


def sr_tune_reset() -> None:
    load_library().sr_tune_reset()

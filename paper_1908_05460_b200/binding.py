"""Thin ctypes binding of libgaconv.so: same names as the C ABI, argument marshalling only.

PyTorch supplies device memory (tensor.data_ptr()) and streams; every step of the path runs inside
the library's CUDA kernels.  Loading fails loudly when the library has not been built: there is no
CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .layers import ConvLayer

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libgaconv.so")

OK = 0
ERR_NULL_POINTER, ERR_BAD_DESC, ERR_UNSUPPORTED, ERR_MISALIGNED, ERR_WORKSPACE_TOO_SMALL, ERR_CUDA, ERR_TIMEOUT = range(1, 8)
F32, BF16 = 0, 1
X_NHWC, X_NCHW = 0, 1
DY_NKPQ, DY_NPQK = 0, 1
DW_KRSC, DW_KCRS, DW_RSCK = 0, 1, 2
METHOD_EXACT, METHOD_ZERO, METHOD_RANDOM, METHOD_TOP1, METHOD_TOPK = -1, 0, 1, 2, 3
MAX_TOPK = 16
MATH_DEFAULT, MATH_TF32 = 0, 1
ALGO_AUTO, ALGO_DIRECT, ALGO_TENSOR = 0, 1, 2
SCHED_EVERY_4TH_LAYER, SCHED_ALT_LAYER_ALT_BATCH, SCHED_ALL_LAYERS_EVERY_4TH_BATCH, SCHED_LAYER2_ALT_BATCH, \
    SCHED_SEEDED_FRACTION_ALT_BATCH = range(5)

EXPORTS = [
    "gaconv_status_string", "gaconv_launch_count", "gaconv_workspace_size", "gaconv_workspace_init", "gaconv_dw_exact",
    "gaconv_dw_approx", "gaconv_approx_select", "gaconv_dw_from_host", "gaconv_dw_from_host_async", "gaconv_poll_async_status",
    "gaconv_schedule_create", "gaconv_schedule_method", "gaconv_schedule_run_layer", "gaconv_schedule_run_step", "gaconv_schedule_destroy",
    "gaconv_dw_exact_static", "gaconv_static_scratch_bytes", "gaconv_poll_async_status_static", "gaconv_approx_select_topk",
]


class ConvDesc(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32)] + \
        [(f, ctypes.c_int32) for f in ("n", "c", "h", "w", "k", "r", "s", "stride_h", "stride_w", "pad_h", "pad_w",
                                       "in_dtype", "x_layout", "dy_layout", "dw_layout", "math", "algo", "topk", "sm_budget")] + \
        [("alpha", ctypes.c_float), ("rand_std", ctypes.c_float),
         ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class GaconvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


_lib = None


def load():
    """Load libgaconv.so; raises if it is missing (build it with paper_1908_05460_b200/build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libgaconv.so is not built: run `python -m paper_1908_05460_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, u64, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_uint64, ctypes.c_size_t
    dp = ctypes.POINTER(ConvDesc)
    lib.gaconv_status_string.restype = ctypes.c_char_p
    lib.gaconv_status_string.argtypes = [ctypes.c_int]
    lib.gaconv_launch_count.restype = ctypes.c_uint64
    lib.gaconv_launch_count.argtypes = []
    lib.gaconv_workspace_size.argtypes = [dp, i32, ctypes.POINTER(sz)]
    lib.gaconv_workspace_init.argtypes = [vp, sz, vp]
    lib.gaconv_dw_exact.argtypes = [vp, vp, vp, dp, vp]
    lib.gaconv_dw_exact_static.argtypes = [vp, vp, vp, dp, vp]
    lib.gaconv_static_scratch_bytes.restype = sz
    lib.gaconv_static_scratch_bytes.argtypes = []
    lib.gaconv_dw_approx.argtypes = [i32, vp, vp, vp, dp, u64, vp]
    lib.gaconv_approx_select.argtypes = [vp, vp, vp, vp, dp, vp]
    lib.gaconv_dw_from_host.argtypes = [i32, vp, vp, vp, vp, vp, vp, dp, u64, vp]
    lib.gaconv_dw_from_host_async.argtypes = [i32, vp, vp, vp, vp, vp, vp, dp, u64, vp]
    lib.gaconv_poll_async_status.argtypes = [dp, vp]
    lib.gaconv_poll_async_status_static.argtypes = [vp]
    lib.gaconv_approx_select_topk.argtypes = [vp, vp, vp, dp, vp]
    lib.gaconv_schedule_create.argtypes = [ctypes.POINTER(vp), i32, i32, i32, ctypes.c_double, u64]
    lib.gaconv_schedule_method.argtypes = [vp, i32, ctypes.c_int64]
    lib.gaconv_schedule_method.restype = i32
    lib.gaconv_schedule_run_layer.argtypes = [vp, i32, ctypes.c_int64, vp, vp, vp, dp, vp]
    lib.gaconv_schedule_run_step.argtypes = [vp, ctypes.c_int64, i32, ctypes.POINTER(vp), ctypes.POINTER(vp), ctypes.POINTER(vp),
                                             ctypes.POINTER(dp), i32, vp]
    lib.gaconv_schedule_destroy.argtypes = [vp]
    lib.gaconv_schedule_destroy.restype = None
    _lib = lib
    return lib


def status_string(status: int) -> str:
    return load().gaconv_status_string(status).decode()


def gaconv_launch_count() -> int:
    return int(load().gaconv_launch_count())


def _check(status: int, where: str):
    if status != OK:
        raise GaconvError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


def make_desc(layer: ConvLayer, dtype: torch.dtype, *, x_layout=X_NHWC, dw_layout=DW_KRSC, alpha=1.0,
              rand_std=1.0 / 128, math=MATH_DEFAULT, algo=ALGO_AUTO, topk=1, sm_budget=0, dy_layout=DY_NKPQ) -> ConvDesc:
    d = ConvDesc()
    d.struct_size = ctypes.sizeof(ConvDesc)
    d.n, d.c, d.h, d.w, d.k, d.r, d.s = layer.n, layer.c, layer.h, layer.w, layer.k, layer.r, layer.s
    d.stride_h = d.stride_w = layer.stride
    d.pad_h = d.pad_w = layer.pad
    d.in_dtype = BF16 if dtype == torch.bfloat16 else F32
    d.x_layout, d.dy_layout, d.dw_layout = x_layout, dy_layout, dw_layout
    d.math, d.algo, d.topk, d.sm_budget = math, algo, topk, sm_budget
    d.alpha, d.rand_std = alpha, rand_std
    d.workspace, d.workspace_bytes = None, 0
    return d


def gaconv_workspace_size(desc: ConvDesc, method: int) -> int:
    out = ctypes.c_size_t(0)
    _check(load().gaconv_workspace_size(ctypes.byref(desc), method, ctypes.byref(out)), "gaconv_workspace_size")
    return out.value


def gaconv_workspace_init(workspace, nbytes: int, stream=None):
    _check(load().gaconv_workspace_init(_ptr(workspace), nbytes, _stream(stream)), "gaconv_workspace_init")


def attach_workspace(desc: ConvDesc, methods=(METHOD_EXACT, METHOD_TOP1, METHOD_TOPK), device="cuda") -> torch.Tensor:
    """Allocate (with torch) and initialise a workspace large enough for `methods`; returns the tensor
    that owns the memory -- keep it alive as long as the descriptor is used."""
    usable = [m for m in methods if m != METHOD_TOPK or 1 <= desc.topk <= MAX_TOPK]
    need = max(gaconv_workspace_size(desc, m) for m in usable)
    ws = torch.empty(need, dtype=torch.uint8, device=device)
    gaconv_workspace_init(ws, need)
    desc.workspace, desc.workspace_bytes = ws.data_ptr(), need
    return ws


def gaconv_dw_exact(x, dy, dw, desc: ConvDesc, stream=None):
    _check(load().gaconv_dw_exact(_ptr(x), _ptr(dy), _ptr(dw), ctypes.byref(desc), _stream(stream)), "gaconv_dw_exact")


def gaconv_dw_exact_static(x, dy, dw, desc: ConvDesc, stream=None):
    """Exact dW for callers that cannot allocate: scratch lives in a fixed array inside the library
    (gaconv_static_scratch_bytes() per GPU); desc.workspace is ignored.  Raises GaconvError with
    ERR_WORKSPACE_TOO_SMALL when the problem needs more scratch than that array holds."""
    _check(load().gaconv_dw_exact_static(_ptr(x), _ptr(dy), _ptr(dw), ctypes.byref(desc), _stream(stream)),
           "gaconv_dw_exact_static")


def gaconv_static_scratch_bytes() -> int:
    return int(load().gaconv_static_scratch_bytes())


def gaconv_dw_approx(method: int, x, dy, dw, desc: ConvDesc, seed: int = 0, stream=None):
    _check(load().gaconv_dw_approx(method, _ptr(x), _ptr(dy), _ptr(dw), ctypes.byref(desc), seed, _stream(stream)),
           "gaconv_dw_approx")


def gaconv_approx_select(dy, idx, sum_, dy_sparse, desc: ConvDesc, stream=None):
    _check(load().gaconv_approx_select(_ptr(dy), _ptr(idx), _ptr(sum_), _ptr(dy_sparse), ctypes.byref(desc),
                                       _stream(stream)), "gaconv_approx_select")


def gaconv_approx_select_topk(dy, idx, sum_, desc: ConvDesc, stream=None):
    _check(load().gaconv_approx_select_topk(_ptr(dy), _ptr(idx), _ptr(sum_), ctypes.byref(desc), _stream(stream)),
           "gaconv_approx_select_topk")


def gaconv_dw_from_host(method: int, x_host, dy_host, dw_host, x_dev, dy_dev, dw_dev, desc: ConvDesc, seed: int = 0,
                        stream=None):
    _check(load().gaconv_dw_from_host(method, _ptr(x_host), _ptr(dy_host), _ptr(dw_host), _ptr(x_dev), _ptr(dy_dev),
                                      _ptr(dw_dev), ctypes.byref(desc), seed, _stream(stream)), "gaconv_dw_from_host")


def gaconv_dw_from_host_async(method: int, x_host, dy_host, dw_host, x_dev, dy_dev, dw_dev, desc: ConvDesc, seed: int = 0,
                              stream=None):
    _check(load().gaconv_dw_from_host_async(method, _ptr(x_host), _ptr(dy_host), _ptr(dw_host), _ptr(x_dev), _ptr(dy_dev),
                                            _ptr(dw_dev), ctypes.byref(desc), seed, _stream(stream)), "gaconv_dw_from_host_async")


def gaconv_poll_async_status(desc: ConvDesc, stream=None) -> int:
    return load().gaconv_poll_async_status(ctypes.byref(desc), _stream(stream))


def gaconv_poll_async_status_static(stream=None) -> int:
    return load().gaconv_poll_async_status_static(_stream(stream))


class Schedule:
    """Owner of a gaconv_schedule_t (host object)."""

    def __init__(self, num_layers: int, kind: int, method: int = METHOD_TOP1, fraction: float = 0.0, seed: int = 0):
        self._h = ctypes.c_void_p()
        _check(load().gaconv_schedule_create(ctypes.byref(self._h), num_layers, kind, method, fraction, seed),
               "gaconv_schedule_create")
        self.num_layers = num_layers

    def method(self, layer: int, step: int) -> int:
        return load().gaconv_schedule_method(self._h, layer, step)

    def run_layer(self, layer: int, step: int, x, dy, dw, desc: ConvDesc, stream=None):
        _check(load().gaconv_schedule_run_layer(self._h, layer, step, _ptr(x), _ptr(dy), _ptr(dw), ctypes.byref(desc),
                                                _stream(stream)), "gaconv_schedule_run_layer")

    def pack_step(self, xs, dys, dws, descs):
        """Marshal the per-layer arrays of run_step once (the tensors and descriptors must stay alive)."""
        n = len(descs)
        VP, DP = ctypes.c_void_p * n, ctypes.POINTER(ConvDesc) * n
        return (n, VP(*[_ptr(t) for t in xs]), VP(*[_ptr(t) for t in dys]), VP(*[_ptr(t) for t in dws]),
                DP(*[ctypes.pointer(d) for d in descs]))

    def run_step(self, step: int, packed, lanes: int = 4, stream=None):
        n, xs, dys, dws, ds = packed
        _check(load().gaconv_schedule_run_step(self._h, step, n, xs, dys, dws, ds, lanes, _stream(stream)),
               "gaconv_schedule_run_step")

    def close(self):
        if self._h:
            load().gaconv_schedule_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

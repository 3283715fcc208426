"""ctypes binding of libsasq_b200.so.  Same names as include/sasq.h.

Every function takes torch CUDA tensors (used purely as device memory), checks
dtype / device / contiguity, and passes raw pointers and sizes to the library on
the current torch stream.  A non-zero status raises SasqError.  If the shared
library is missing or cannot be loaded, import of this module's functions fails
loudly: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os

import torch

__all__ = [
    "SasqError", "SASQ_F16", "SASQ_BF16", "library_path", "load_library", "sasq_status_string",
    "sasq_fakequant_fwd", "sasq_fakequant_bwd_workspace", "sasq_fakequant_bwd", "sasq_fakequant_fwd_bwd",
    "sasq_fakequant_multi_workspace", "sasq_fakequant_fwd_bwd_multi", "sasq_static_w8a8_linear_workspace",
    "sasq_static_w8a8_linear", "sasq_device_status", "QDesc", "sasq_absmax_scale_workspace", "sasq_absmax_scale",
    "sasq_quantize_weight", "sasq_fakequant_fwd_bwd_static", "sasq_static_w8a8_linear_tiles",
    "sasq_fakequant_per_channel_workspace", "sasq_fakequant_fwd_bwd_per_channel",
    "sasq_fakequant_fwd_bwd_ablation", "sasq_adamw_scales", "SASQ_FULL_OPERATOR", "SASQ_WITHOUT_ROUND",
    "SASQ_WITHOUT_CLAMP", "sasq_dynamic_w8a8_linear_workspace", "sasq_dynamic_w8a8_linear", "sasq_debug_set_wait_limit", "PcDesc", "sasq_fakequant_per_channel_multi_workspace",
    "sasq_fakequant_fwd_bwd_per_channel_multi", "sasq_static_w8a8_linear_per_channel_workspace",
    "sasq_static_w8a8_linear_per_channel", "sasq_static_w8a8_linear_grouped_workspace",
    "sasq_static_w8a8_linear_grouped", "sasq_fakequant_linear_fp_weights_workspace",
    "sasq_fakequant_linear_fp_weights", "sasq_absmax_scale_per_channel", "sasq_running_mean", "LinearDesc", "sasq_static_w8a8_linear_multi_workspace",
    "sasq_static_w8a8_linear_multi", "sasq_static_w8a8_linear_multi_launches", "sasq_set_gang_launch",
    "sasq_debug_int8_issue_rate", "LinearProblems", "QuantTensors",
]

SASQ_F16 = 0
SASQ_BF16 = 1
SASQ_FULL_OPERATOR = 0
SASQ_WITHOUT_ROUND = 1
SASQ_WITHOUT_CLAMP = 2


_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libsasq_b200.so")
_lib = None


class SasqError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: {sasq_status_string(status)} (status {status})")


class QDesc(ctypes.Structure):
    """Mirror of sasq_qdesc_t."""
    _fields_ = [("x", ctypes.c_void_p), ("grad_y", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("grad_x", ctypes.c_void_p), ("numel", ctypes.c_int64), ("scale_index", ctypes.c_int32),
                ("reserved", ctypes.c_int32)]


class PcDesc(ctypes.Structure):
    """Mirror of sasq_pcdesc_t."""
    _fields_ = [("x", ctypes.c_void_p), ("grad_y", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("grad_x", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("grad_scales", ctypes.c_void_p),
                ("T", ctypes.c_int64), ("K", ctypes.c_int64), ("reserved", ctypes.c_int64)]


class LinearDesc(ctypes.Structure):
    """Mirror of sasq_linear_desc_t."""
    _fields_ = [("x", ctypes.c_void_p), ("w", ctypes.c_void_p), ("w_scale", ctypes.c_void_p),
                ("x_scale", ctypes.c_void_p), ("bias", ctypes.c_void_p), ("y", ctypes.c_void_p),
                ("T", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64)]


def library_path() -> str:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (python -m paper_2512_14481_b200.build)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2512_14481_b200.build` "
                           "(there is no fallback path)")
    L = ctypes.CDLL(_LIB_PATH)
    vp, i64, i32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_size_t
    L.sasq_status_string.restype = ctypes.c_char_p
    L.sasq_status_string.argtypes = [i32]
    L.sasq_fakequant_fwd.restype = i32
    L.sasq_fakequant_fwd.argtypes = [vp, vp, i64, i32, vp, i32, vp]
    L.sasq_fakequant_bwd_workspace.restype = sz
    L.sasq_fakequant_bwd_workspace.argtypes = [i64]
    L.sasq_fakequant_bwd.restype = i32
    L.sasq_fakequant_bwd.argtypes = [vp, vp, vp, vp, i32, i64, i32, vp, i32, vp, sz, vp]
    L.sasq_fakequant_fwd_bwd.restype = i32
    L.sasq_fakequant_fwd_bwd.argtypes = [vp, vp, vp, vp, vp, i32, i64, i32, vp, i32, vp, sz, vp]
    L.sasq_fakequant_fwd_bwd_static.restype = i32
    L.sasq_fakequant_fwd_bwd_static.argtypes = [vp, vp, vp, vp, vp, i32, i64, i32, vp, i32, vp]
    L.sasq_fakequant_multi_workspace.restype = sz
    L.sasq_fakequant_multi_workspace.argtypes = [i32]
    L.sasq_fakequant_fwd_bwd_multi.restype = i32
    L.sasq_fakequant_fwd_bwd_multi.argtypes = [ctypes.POINTER(QDesc), i32, vp, vp, i32, i32, i32, i32, vp, sz, vp]
    L.sasq_static_w8a8_linear_workspace.restype = sz
    L.sasq_static_w8a8_linear_workspace.argtypes = [i64, i64, i64]
    L.sasq_static_w8a8_linear.restype = i32
    L.sasq_static_w8a8_linear.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, sz, vp]
    L.sasq_fakequant_fwd_bwd_ablation.restype = i32
    L.sasq_fakequant_fwd_bwd_ablation.argtypes = [vp, vp, vp, vp, vp, i32, i64, i32, vp, i32, i32, vp, sz, vp]
    f32 = ctypes.c_float
    L.sasq_adamw_scales.restype = i32
    L.sasq_adamw_scales.argtypes = [vp, vp, vp, vp, i32, i32, f32, f32, f32, f32, f32, vp]
    L.sasq_fakequant_per_channel_workspace.restype = sz
    L.sasq_fakequant_per_channel_workspace.argtypes = [i64, i64]
    L.sasq_fakequant_fwd_bwd_per_channel.restype = i32
    L.sasq_fakequant_fwd_bwd_per_channel.argtypes = [vp, vp, vp, vp, vp, i32, i64, i64, i32, vp, i32, vp, sz, vp]
    L.sasq_static_w8a8_linear_per_channel_workspace.restype = sz
    L.sasq_static_w8a8_linear_per_channel_workspace.argtypes = [i64, i64, i64]
    L.sasq_static_w8a8_linear_per_channel.restype = i32
    L.sasq_static_w8a8_linear_per_channel.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, sz, vp]
    L.sasq_dynamic_w8a8_linear_workspace.restype = sz
    L.sasq_dynamic_w8a8_linear_workspace.argtypes = [i64, i64, i64]
    L.sasq_dynamic_w8a8_linear.restype = i32
    L.sasq_dynamic_w8a8_linear.argtypes = [vp, vp, vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, sz, vp]
    L.sasq_fakequant_per_channel_multi_workspace.restype = sz
    L.sasq_fakequant_per_channel_multi_workspace.argtypes = [i64]
    L.sasq_fakequant_fwd_bwd_per_channel_multi.restype = i32
    L.sasq_fakequant_fwd_bwd_per_channel_multi.argtypes = [ctypes.POINTER(PcDesc), i32, i32, i32, i32, vp, sz, vp]
    L.sasq_debug_set_wait_limit.restype = ctypes.c_longlong
    L.sasq_debug_set_wait_limit.argtypes = [ctypes.c_longlong]
    L.sasq_fakequant_linear_fp_weights_workspace.restype = sz
    L.sasq_fakequant_linear_fp_weights_workspace.argtypes = [i64, i64, i64]
    L.sasq_fakequant_linear_fp_weights.restype = i32
    L.sasq_fakequant_linear_fp_weights.argtypes = [vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, vp, sz, vp]
    L.sasq_static_w8a8_linear_grouped_workspace.restype = sz
    L.sasq_static_w8a8_linear_grouped_workspace.argtypes = [i64, i64, i64]
    L.sasq_static_w8a8_linear_grouped.restype = i32
    L.sasq_static_w8a8_linear_grouped.argtypes = [vp, vp, vp, vp, i64, vp, vp, i64, i64, i64, i32, i32, vp, sz, vp]
    L.sasq_static_w8a8_linear_multi_workspace.restype = sz
    L.sasq_static_w8a8_linear_multi_workspace.argtypes = [i32, ctypes.POINTER(LinearDesc)]
    L.sasq_static_w8a8_linear_multi.restype = i32
    L.sasq_static_w8a8_linear_multi.argtypes = [i32, ctypes.POINTER(LinearDesc), i32, i32, vp, sz, vp]
    L.sasq_static_w8a8_linear_multi_launches.restype = i32
    L.sasq_static_w8a8_linear_multi_launches.argtypes = [i32, ctypes.POINTER(LinearDesc), i32]
    L.sasq_static_w8a8_linear_tiles.restype = i32
    L.sasq_static_w8a8_linear_tiles.argtypes = [i64, i64, i32, i32, ctypes.POINTER(ctypes.c_int32), i32]
    L.sasq_device_status.restype = i32
    L.sasq_device_status.argtypes = [vp]
    L.sasq_absmax_scale_workspace.restype = sz
    L.sasq_absmax_scale_workspace.argtypes = [i64]
    L.sasq_absmax_scale.restype = i32
    L.sasq_absmax_scale.argtypes = [vp, i64, i32, i32, vp, vp, sz, vp]
    L.sasq_quantize_weight.restype = i32
    L.sasq_quantize_weight.argtypes = [vp, vp, vp, i64, i64, i32, vp]
    _lib = L
    return L


def sasq_status_string(status: int) -> str:
    return load_library().sasq_status_string(int(status)).decode()


# ---------------------------------------------------------------------------
# marshalling helpers
# ---------------------------------------------------------------------------
def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float16:
        return SASQ_F16
    if t.dtype == torch.bfloat16:
        return SASQ_BF16
    raise TypeError(f"expected float16 or bfloat16, got {t.dtype}")


def _dev(t, name: str, dtype=None):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise TypeError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")
    return t


def _ptr(t) -> int | None:
    return None if t is None else t.data_ptr()


def _stream(stream) -> int:
    """None: torch's current stream; a torch stream; or a raw cudaStream_t handle as an int (the cheapest to pass)."""
    if isinstance(stream, int):
        return stream
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


# SASQ_DEBUG_STATUS=1 in the environment: every call through this binding also synchronises and reads the sticky
# device status word, so that a device-detected problem (a bad factor, a bounded wait that gave up) raises at the
# call that caused it instead of waiting for the caller's next sasq_device_status().  For tests and debugging only.
_DEBUG_STATUS = os.environ.get("SASQ_DEBUG_STATUS", "0") not in ("", "0")


def _check(status: int, where: str):
    if status != 0:
        raise SasqError(status, where)
    if _DEBUG_STATUS:
        dev_status = int(load_library().sasq_device_status(_stream(None)))
        if dev_status != 0:
            raise SasqError(dev_status, where + " (device status)")


def _nbytes(t) -> int:
    return 0 if t is None else t.numel() * t.element_size()


# ---------------------------------------------------------------------------
# the entry points
# ---------------------------------------------------------------------------
def sasq_fakequant_fwd(x: torch.Tensor, y: torch.Tensor, scale: torch.Tensor, bits: int = 8, stream=None) -> None:
    _dev(x, "x"); _dev(y, "y", x.dtype); _dev(scale, "scale", torch.float32)
    if y.numel() != x.numel():
        raise ValueError("y must have as many elements as x")
    _check(load_library().sasq_fakequant_fwd(_ptr(x), _ptr(y), x.numel(), _dt(x), _ptr(scale), int(bits),
                                             _stream(stream)), "sasq_fakequant_fwd")


def sasq_fakequant_bwd_workspace(numel: int) -> int:
    return int(load_library().sasq_fakequant_bwd_workspace(int(numel)))


def sasq_fakequant_bwd(x, grad_y, grad_x, grad_scale, scale, workspace, bits: int = 8, accumulate: bool = False,
                       stream=None) -> None:
    _dev(x, "x"); _dev(grad_y, "grad_y", x.dtype); _dev(grad_x, "grad_x", x.dtype)
    _dev(grad_scale, "grad_scale", torch.float32); _dev(scale, "scale", torch.float32); _dev(workspace, "workspace")
    if grad_y.numel() != x.numel() or grad_x.numel() != x.numel():
        raise ValueError("grad_y and grad_x must have as many elements as x")
    _check(load_library().sasq_fakequant_bwd(_ptr(x), _ptr(grad_y), _ptr(grad_x), _ptr(grad_scale), int(bool(accumulate)),
                                             x.numel(), _dt(x), _ptr(scale), int(bits), _ptr(workspace),
                                             _nbytes(workspace), _stream(stream)), "sasq_fakequant_bwd")


def sasq_fakequant_fwd_bwd(x, grad_y, y, grad_x, grad_scale, scale, workspace, bits: int = 8,
                           accumulate: bool = False, stream=None) -> None:
    _dev(x, "x"); _dev(grad_y, "grad_y", x.dtype); _dev(y, "y", x.dtype); _dev(grad_x, "grad_x", x.dtype)
    _dev(grad_scale, "grad_scale", torch.float32); _dev(scale, "scale", torch.float32); _dev(workspace, "workspace")
    if grad_y.numel() != x.numel() or grad_x.numel() != x.numel() or y.numel() != x.numel():
        raise ValueError("grad_y, y and grad_x must have as many elements as x")
    _check(load_library().sasq_fakequant_fwd_bwd(_ptr(x), _ptr(grad_y), _ptr(y), _ptr(grad_x), _ptr(grad_scale),
                                                 int(bool(accumulate)), x.numel(), _dt(x), _ptr(scale), int(bits),
                                                 _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sasq_fakequant_fwd_bwd")


def sasq_fakequant_multi_workspace(n_tensors: int) -> int:
    return int(load_library().sasq_fakequant_multi_workspace(int(n_tensors)))


class QuantTensors:
    """The descriptor table of a sasq_fakequant_fwd_bwd_multi call, marshalled once (see LinearProblems)."""

    def __init__(self, tensors):
        self.tensors = list(tensors)
        n = len(self.tensors)
        self.descs = (QDesc * max(n, 1))()
        dt = None
        for i, (x, gy, y, gx, idx) in enumerate(self.tensors):
            _dev(x, "x")
            for name, t in (("grad_y", gy), ("y", y), ("grad_x", gx)):
                if t is not None:
                    _dev(t, name, x.dtype)
                    if t.numel() != x.numel():
                        raise ValueError(f"{name} must have as many elements as x")
            if dt is None:
                dt = _dt(x)
            elif dt != _dt(x):
                raise TypeError("all tensors of one call must share a dtype")
            self.descs[i] = QDesc(_ptr(x), _ptr(gy), _ptr(y), _ptr(gx), x.numel(), int(idx), 0)
        self.dt = SASQ_BF16 if dt is None else dt
        self.count = n


def sasq_fakequant_fwd_bwd_multi(tensors, scales, grad_scales, workspace, bits: int = 8, accumulate: bool = False,
                                 stream=None) -> None:
    """tensors: sequence of (x, grad_y | None, y | None, grad_x | None, scale_index), or a QuantTensors made from one."""
    prepared = tensors if isinstance(tensors, QuantTensors) else QuantTensors(tensors)
    _dev(scales, "scales", torch.float32)
    if grad_scales is not None:
        _dev(grad_scales, "grad_scales", torch.float32)
    if workspace is not None:
        _dev(workspace, "workspace")
    _check(load_library().sasq_fakequant_fwd_bwd_multi(prepared.descs, prepared.count, _ptr(scales), _ptr(grad_scales),
                                                       scales.numel(), int(bool(accumulate)), prepared.dt,
                                                       int(bits), _ptr(workspace), _nbytes(workspace),
                                                       _stream(stream)), "sasq_fakequant_fwd_bwd_multi")


def sasq_fakequant_fwd_bwd_ablation(x, grad_y, y, grad_x, grad_scale, scale, workspace, variant: int, bits: int = 8,
                                    accumulate: bool = False, stream=None) -> None:
    """The fused pass with Table 3's "w/o round" / "w/o clamp" ablations (variant = SASQ_WITHOUT_*)."""
    _dev(x, "x"); _dev(grad_y, "grad_y", x.dtype); _dev(y, "y", x.dtype); _dev(grad_x, "grad_x", x.dtype)
    _dev(grad_scale, "grad_scale", torch.float32); _dev(scale, "scale", torch.float32); _dev(workspace, "workspace")
    if grad_y.numel() != x.numel() or grad_x.numel() != x.numel() or y.numel() != x.numel():
        raise ValueError("grad_y, y and grad_x must have as many elements as x")
    _check(load_library().sasq_fakequant_fwd_bwd_ablation(_ptr(x), _ptr(grad_y), _ptr(y), _ptr(grad_x),
                                                          _ptr(grad_scale), int(bool(accumulate)), x.numel(), _dt(x),
                                                          _ptr(scale), int(bits), int(variant), _ptr(workspace),
                                                          _nbytes(workspace), _stream(stream)),
           "sasq_fakequant_fwd_bwd_ablation")


def sasq_adamw_scales(scales, grad_scales, exp_avg, exp_avg_sq, step: int, lr: float = 2e-4, beta1: float = 0.9,
                      beta2: float = 0.999, eps: float = 1e-8, weight_decay: float = 0.01, stream=None) -> None:
    """One AdamW step on the factors, in place (scales, exp_avg, exp_avg_sq: fp32 CUDA tensors of one size)."""
    for name, t in (("scales", scales), ("grad_scales", grad_scales), ("exp_avg", exp_avg), ("exp_avg_sq", exp_avg_sq)):
        _dev(t, name, torch.float32)
        if t.numel() != scales.numel():
            raise ValueError(f"{name} must have as many elements as scales")
    _check(load_library().sasq_adamw_scales(_ptr(scales), _ptr(grad_scales), _ptr(exp_avg), _ptr(exp_avg_sq),
                                            scales.numel(), int(step), float(lr), float(beta1), float(beta2),
                                            float(eps), float(weight_decay), _stream(stream)), "sasq_adamw_scales")


def sasq_fakequant_per_channel_workspace(T: int, K: int) -> int:
    return int(load_library().sasq_fakequant_per_channel_workspace(int(T), int(K)))


def sasq_fakequant_fwd_bwd_per_channel(x, grad_y, y, grad_x, grad_scales, scales, workspace, bits: int = 8,
                                       accumulate: bool = False, stream=None) -> None:
    """x [T, K] with one factor per column: scales [K], grad_scales [K]; y or (grad_y, grad_x) may be None."""
    _dev(x, "x"); _dev(scales, "scales", torch.float32)
    if x.dim() != 2 or scales.numel() != x.shape[1]:
        raise ValueError("x must be [T, K] and scales [K]")
    for name, t in (("grad_y", grad_y), ("y", y), ("grad_x", grad_x)):
        if t is not None:
            _dev(t, name, x.dtype)
            if tuple(t.shape) != tuple(x.shape):
                raise ValueError(f"{name} must have the shape of x")
    if grad_scales is not None:
        _dev(grad_scales, "grad_scales", torch.float32)
        if grad_scales.numel() != x.shape[1]:
            raise ValueError("grad_scales must be [K]")
    if workspace is not None:
        _dev(workspace, "workspace")
    _check(load_library().sasq_fakequant_fwd_bwd_per_channel(_ptr(x), _ptr(grad_y), _ptr(y), _ptr(grad_x),
                                                             _ptr(grad_scales), int(bool(accumulate)), x.shape[0],
                                                             x.shape[1], _dt(x), _ptr(scales), int(bits),
                                                             _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sasq_fakequant_fwd_bwd_per_channel")


def sasq_fakequant_per_channel_multi_workspace(total_K: int) -> int:
    return int(load_library().sasq_fakequant_per_channel_multi_workspace(int(total_K)))


def sasq_fakequant_fwd_bwd_per_channel_multi(tensors, workspace, bits: int = 8, accumulate: bool = False,
                                             stream=None) -> None:
    """tensors: sequence of (x [T, K], grad_y | None, y | None, grad_x | None, scales [K], grad_scales [K] | None)."""
    n = len(tensors)
    descs = (PcDesc * max(n, 1))()
    dt = None
    for i, (x, gy, y, gx, sc, gs) in enumerate(tensors):
        _dev(x, "x"); _dev(sc, "scales", torch.float32)
        if x.dim() != 2 or sc.numel() != x.shape[1]:
            raise ValueError("x must be [T, K] and scales [K]")
        for name, t in (("grad_y", gy), ("y", y), ("grad_x", gx)):
            if t is not None:
                _dev(t, name, x.dtype)
                if tuple(t.shape) != tuple(x.shape):
                    raise ValueError(f"{name} must have the shape of x")
        if gs is not None:
            _dev(gs, "grad_scales", torch.float32)
        if dt is None:
            dt = _dt(x)
        elif dt != _dt(x):
            raise TypeError("all tensors of one call must share a dtype")
        descs[i] = PcDesc(_ptr(x), _ptr(gy), _ptr(y), _ptr(gx), _ptr(sc), _ptr(gs), x.shape[0], x.shape[1], 0)
    if workspace is not None:
        _dev(workspace, "workspace")
    _check(load_library().sasq_fakequant_fwd_bwd_per_channel_multi(descs, n, int(bool(accumulate)),
                                                                   SASQ_BF16 if dt is None else dt, int(bits),
                                                                   _ptr(workspace), _nbytes(workspace),
                                                                   _stream(stream)),
           "sasq_fakequant_fwd_bwd_per_channel_multi")


def sasq_static_w8a8_linear_workspace(T: int, N: int, K: int) -> int:
    return int(load_library().sasq_static_w8a8_linear_workspace(int(T), int(N), int(K)))


def sasq_static_w8a8_linear(x, w, w_scale, x_scale, y, bias=None, acc_out=None, workspace=None, bits: int = 8,
                            stream=None) -> None:
    """x [T, K] fp16/bf16, w [N, K] int8, w_scale [N] fp32, x_scale [1] fp32, y [T, N]."""
    _dev(x, "x"); _dev(w, "w", torch.int8); _dev(w_scale, "w_scale", torch.float32)
    _dev(x_scale, "x_scale", torch.float32); _dev(y, "y", x.dtype)
    if bias is not None:
        _dev(bias, "bias", x.dtype)
    if acc_out is not None:
        _dev(acc_out, "acc_out", torch.int32)
    if workspace is not None:
        _dev(workspace, "workspace")
    if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1]:
        raise ValueError("x must be [T, K] and w [N, K]")
    T, K = x.shape
    N = w.shape[0]
    if tuple(y.shape) != (T, N) or w_scale.numel() != N or (bias is not None and bias.numel() != N):
        raise ValueError("y must be [T, N], w_scale and bias [N]")
    if acc_out is not None and tuple(acc_out.shape) != (T, N):
        raise ValueError("acc_out must be [T, N]")
    _check(load_library().sasq_static_w8a8_linear(_ptr(x), _ptr(w), _ptr(w_scale), _ptr(x_scale), _ptr(bias), _ptr(y),
                                                  _ptr(acc_out), T, N, K, _dt(x), int(bits), _ptr(workspace),
                                                  _nbytes(workspace), _stream(stream)), "sasq_static_w8a8_linear")


def sasq_fakequant_linear_fp_weights_workspace(T: int, N: int, K: int) -> int:
    return int(load_library().sasq_fakequant_linear_fp_weights_workspace(int(T), int(N), int(K)))


def sasq_fakequant_linear_fp_weights(x, w, x_scale, y, bias=None, workspace=None, bits: int = 8, stream=None) -> None:
    """Table 3's "FP weights" form: fake-quantized activations times 16-bit weights; x [T, K], w [N, K], y [T, N]."""
    _dev(x, "x"); _dev(w, "w", x.dtype); _dev(x_scale, "x_scale", torch.float32); _dev(y, "y", x.dtype)
    if bias is not None:
        _dev(bias, "bias", x.dtype)
    if workspace is not None:
        _dev(workspace, "workspace")
    if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1]:
        raise ValueError("x must be [T, K] and w [N, K]")
    T, K = x.shape
    N = w.shape[0]
    if tuple(y.shape) != (T, N) or (bias is not None and bias.numel() != N):
        raise ValueError("y must be [T, N] and bias [N]")
    _check(load_library().sasq_fakequant_linear_fp_weights(_ptr(x), _ptr(w), _ptr(x_scale), _ptr(bias), _ptr(y), T, N, K,
                                                           _dt(x), int(bits), _ptr(workspace), _nbytes(workspace),
                                                           _stream(stream)), "sasq_fakequant_linear_fp_weights")


def sasq_static_w8a8_linear_grouped_workspace(T: int, N: int, K: int) -> int:
    return int(load_library().sasq_static_w8a8_linear_grouped_workspace(int(T), int(N), int(K)))


def sasq_static_w8a8_linear_grouped(x, w, w_scale, s_group, group: int, y, bias=None, workspace=None, bits: int = 8,
                                    stream=None) -> None:
    """Eq. 3: x [T, K], one static factor per group of `group` consecutive channels (s_group [K / group])."""
    _dev(x, "x"); _dev(w, "w", torch.int8); _dev(w_scale, "w_scale", torch.float32)
    _dev(s_group, "s_group", torch.float32); _dev(y, "y", x.dtype)
    if bias is not None:
        _dev(bias, "bias", x.dtype)
    if workspace is not None:
        _dev(workspace, "workspace")
    if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1]:
        raise ValueError("x must be [T, K] and w [N, K]")
    T, K = x.shape
    N = w.shape[0]
    if group <= 0 or K % group != 0 or s_group.numel() != K // group:
        raise ValueError("s_group must hold one factor per group of `group` channels")
    if tuple(y.shape) != (T, N) or w_scale.numel() != N or (bias is not None and bias.numel() != N):
        raise ValueError("y must be [T, N], w_scale and bias [N]")
    _check(load_library().sasq_static_w8a8_linear_grouped(_ptr(x), _ptr(w), _ptr(w_scale), _ptr(s_group), int(group),
                                                          _ptr(bias), _ptr(y), T, N, K, _dt(x), int(bits),
                                                          _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sasq_static_w8a8_linear_grouped")


def _linear_descs(problems):
    """problems: sequence of (x, w, w_scale, x_scale, y) or (x, w, w_scale, x_scale, y, bias)."""
    arr = (LinearDesc * max(1, len(problems)))()
    dt = None
    for i, pr in enumerate(problems):
        x, w, w_scale, x_scale, y = pr[:5]
        bias = pr[5] if len(pr) > 5 else None
        _dev(x, "x"); _dev(w, "w", torch.int8); _dev(w_scale, "w_scale", torch.float32)
        _dev(x_scale, "x_scale", torch.float32); _dev(y, "y", x.dtype)
        if bias is not None:
            _dev(bias, "bias", x.dtype)
        if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1]:
            raise ValueError("x must be [T, K] and w [N, K]")
        T, K = x.shape
        N = w.shape[0]
        if tuple(y.shape) != (T, N) or w_scale.numel() != N or (bias is not None and bias.numel() != N):
            raise ValueError("y must be [T, N], w_scale and bias [N]")
        if dt is None:
            dt = _dt(x)
        elif dt != _dt(x):
            raise ValueError("all problems of one call share the activation dtype")
        arr[i] = LinearDesc(_ptr(x), _ptr(w), _ptr(w_scale), _ptr(x_scale), _ptr(bias), _ptr(y), T, N, K)
    return arr, dt


def sasq_static_w8a8_linear_multi_workspace(shapes) -> int:
    """shapes: sequence of (T, N, K)."""
    arr = (LinearDesc * max(1, len(shapes)))()
    for i, (T, N, K) in enumerate(shapes):
        arr[i].T, arr[i].N, arr[i].K = int(T), int(N), int(K)
    return int(load_library().sasq_static_w8a8_linear_multi_workspace(len(shapes), arr))


class LinearProblems:
    """The descriptor table of a sasq_static_w8a8_linear_multi call, marshalled once: a caller that submits the same
    tensors again and again (a layer's weights and activation buffers) passes this instead of the tuples and skips
    the per-call checks and conversions.  Holds references to the tensors so the pointers stay valid."""

    def __init__(self, problems):
        self.problems = list(problems)
        self.descs, dt = _linear_descs(self.problems)
        self.dt = SASQ_BF16 if dt is None else dt
        self.count = len(self.problems)
        self._ws = None         # (workspace tensor, pointer, bytes) of the last call: checked once per workspace


def sasq_static_w8a8_linear_multi(problems, workspace, bits: int = 8, stream=None) -> None:
    """Independent static W8A8 linears submitted together: a sequence of tuples (see _linear_descs) or a
    LinearProblems made from one."""
    prepared = problems if isinstance(problems, LinearProblems) else LinearProblems(problems)
    ws = prepared._ws
    if ws is None or ws[0] is not workspace:
        _dev(workspace, "workspace")
        ws = prepared._ws = (workspace, _ptr(workspace), _nbytes(workspace))
    _check(load_library().sasq_static_w8a8_linear_multi(prepared.count, prepared.descs, prepared.dt, int(bits),
                                                        ws[1], ws[2], _stream(stream)),
           "sasq_static_w8a8_linear_multi")


def sasq_static_w8a8_linear_multi_launches(shapes, num_pairs: int = 74) -> int:
    """Kernels one sasq_static_w8a8_linear_multi call launches for problems of these (T, N, K) on a device with
    `num_pairs` resident CTA pairs (launch counting; asks the library, touches no device)."""
    arr = (LinearDesc * max(1, len(shapes)))()
    for i, (T, N, K) in enumerate(shapes):
        arr[i].T, arr[i].N, arr[i].K = int(T), int(N), int(K)
    n = int(load_library().sasq_static_w8a8_linear_multi_launches(len(shapes), arr, int(num_pairs)))
    if n < 0:
        raise ValueError("invalid shapes")
    return n


def sasq_static_w8a8_linear_per_channel_workspace(T: int, N: int, K: int) -> int:
    return int(load_library().sasq_static_w8a8_linear_per_channel_workspace(int(T), int(N), int(K)))


def sasq_static_w8a8_linear_per_channel(x, w, w_scale, x_scales, y, bias=None, acc_out=None, workspace=None,
                                        bits: int = 8, stream=None) -> None:
    """x [T, K], x_scales [K] (one static factor per channel, already folded into w), w [N, K] int8, y [T, N]."""
    _dev(x, "x"); _dev(w, "w", torch.int8); _dev(w_scale, "w_scale", torch.float32)
    _dev(x_scales, "x_scales", torch.float32); _dev(y, "y", x.dtype)
    for name, t, dtp in (("bias", bias, x.dtype), ("acc_out", acc_out, torch.int32)):
        if t is not None:
            _dev(t, name, dtp)
    if workspace is not None:
        _dev(workspace, "workspace")
    if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1] or x_scales.numel() != x.shape[1]:
        raise ValueError("x must be [T, K], w [N, K] and x_scales [K]")
    T, K = x.shape
    N = w.shape[0]
    if tuple(y.shape) != (T, N) or w_scale.numel() != N or (bias is not None and bias.numel() != N):
        raise ValueError("y must be [T, N], w_scale and bias [N]")
    _check(load_library().sasq_static_w8a8_linear_per_channel(_ptr(x), _ptr(w), _ptr(w_scale), _ptr(x_scales),
                                                              _ptr(bias), _ptr(y), _ptr(acc_out), T, N, K, _dt(x),
                                                              int(bits), _ptr(workspace), _nbytes(workspace),
                                                              _stream(stream)),
           "sasq_static_w8a8_linear_per_channel")


def sasq_dynamic_w8a8_linear_workspace(T: int, N: int, K: int) -> int:
    return int(load_library().sasq_dynamic_w8a8_linear_workspace(int(T), int(N), int(K)))


def sasq_dynamic_w8a8_linear(x, w, w_scale, y, bias=None, row_scale_out=None, acc_out=None, workspace=None,
                             bits: int = 8, stream=None) -> None:
    """Dynamic per-token W8A8 linear: x [T, K], w [N, K] int8, w_scale [N], y [T, N]; row_scale_out [T] fp32 or None."""
    _dev(x, "x"); _dev(w, "w", torch.int8); _dev(w_scale, "w_scale", torch.float32); _dev(y, "y", x.dtype)
    for name, t, dtp in (("bias", bias, x.dtype), ("row_scale_out", row_scale_out, torch.float32),
                         ("acc_out", acc_out, torch.int32)):
        if t is not None:
            _dev(t, name, dtp)
    if workspace is not None:
        _dev(workspace, "workspace")
    if x.dim() != 2 or w.dim() != 2 or x.shape[1] != w.shape[1]:
        raise ValueError("x must be [T, K] and w [N, K]")
    T, K = x.shape
    N = w.shape[0]
    if tuple(y.shape) != (T, N) or w_scale.numel() != N or (bias is not None and bias.numel() != N):
        raise ValueError("y must be [T, N], w_scale and bias [N]")
    if row_scale_out is not None and row_scale_out.numel() != T:
        raise ValueError("row_scale_out must be [T]")
    if acc_out is not None and tuple(acc_out.shape) != (T, N):
        raise ValueError("acc_out must be [T, N]")
    _check(load_library().sasq_dynamic_w8a8_linear(_ptr(x), _ptr(w), _ptr(w_scale), _ptr(bias), _ptr(y),
                                                   _ptr(row_scale_out), _ptr(acc_out), T, N, K, _dt(x), int(bits),
                                                   _ptr(workspace), _nbytes(workspace), _stream(stream)),
           "sasq_dynamic_w8a8_linear")


def sasq_static_w8a8_linear_tiles(T: int, N: int, num_pairs: int, pair_id: int):
    """Tiles (first row, first column, width) that CTA pair `pair_id` of `num_pairs` walks for a [T, N] output."""
    L = load_library()
    n = L.sasq_static_w8a8_linear_tiles(int(T), int(N), int(num_pairs), int(pair_id), None, 0)
    if n < 0:
        raise ValueError("invalid arguments")
    buf = (ctypes.c_int32 * (3 * max(n, 1)))()
    L.sasq_static_w8a8_linear_tiles(int(T), int(N), int(num_pairs), int(pair_id), buf, n)
    return [(buf[3 * i], buf[3 * i + 1], buf[3 * i + 2]) for i in range(n)]


def sasq_debug_set_wait_limit(cycles: int) -> int:
    """Test hook: clock cycles after which a wait inside the GEMM kernels gives up (negative restores the default)."""
    return int(load_library().sasq_debug_set_wait_limit(int(cycles)))


def sasq_debug_int8_issue_rate(mma_per_pair: int, n_cols: int = 256, stream=None):
    """Measurement aid: back-to-back int8 tensor-core instructions of the GEMM's shape on every CTA pair.
    Returns (integer operations per second of the device, multiply-accumulates per clock per SM)."""
    L = load_library()
    L.sasq_debug_int8_issue_rate.restype = ctypes.c_int
    L.sasq_debug_int8_issue_rate.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.POINTER(ctypes.c_double),
                                             ctypes.POINTER(ctypes.c_double), ctypes.c_void_p]
    ops, mac = ctypes.c_double(0.0), ctypes.c_double(0.0)
    _check(L.sasq_debug_int8_issue_rate(int(mma_per_pair), int(n_cols), ctypes.byref(ops), ctypes.byref(mac),
                                        _stream(stream)), "sasq_debug_int8_issue_rate")
    return float(ops.value), float(mac.value)


def sasq_set_gang_launch(on: bool) -> bool:
    """Launch the linears whose CTAs wait on one another as co-operative grids (the default; safe with several
    streams).  A caller that keeps all linears on one stream may pass False; returns the previous setting."""
    L = load_library()
    L.sasq_set_gang_launch.restype = ctypes.c_int
    L.sasq_set_gang_launch.argtypes = [ctypes.c_int]
    return bool(L.sasq_set_gang_launch(1 if on else 0))


def sasq_device_status(stream=None) -> int:
    """Synchronises the stream; returns and clears the sticky device status (0 = OK)."""
    return int(load_library().sasq_device_status(_stream(stream)))


def sasq_absmax_scale_per_channel(x, scales_out, bits: int = 8, stream=None) -> None:
    """scales_out[k] = max_t |x[t, k]| / Qp (Eq. 1 per channel) of one calibration batch; x [T, K]."""
    _dev(x, "x"); _dev(scales_out, "scales_out", torch.float32)
    if x.dim() != 2 or scales_out.numel() != x.shape[1]:
        raise ValueError("x must be [T, K] and scales_out [K]")
    L = load_library()
    L.sasq_absmax_scale_per_channel.restype = ctypes.c_int
    L.sasq_absmax_scale_per_channel.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                                ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
    _check(L.sasq_absmax_scale_per_channel(_ptr(x), x.shape[0], x.shape[1], _dt(x), int(bits), _ptr(scales_out),
                                           _stream(stream)), "sasq_absmax_scale_per_channel")


def sasq_running_mean(mean, value, count: int, stream=None) -> None:
    """mean <- mean of the first `count` values, given the mean of the first count - 1 and the count-th value."""
    _dev(mean, "mean", torch.float32); _dev(value, "value", torch.float32)
    if mean.numel() != value.numel():
        raise ValueError("mean and value must have the same number of elements")
    L = load_library()
    L.sasq_running_mean.restype = ctypes.c_int
    L.sasq_running_mean.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
    _check(L.sasq_running_mean(_ptr(mean), _ptr(value), mean.numel(), int(count), _stream(stream)), "sasq_running_mean")


def sasq_absmax_scale_workspace(numel: int) -> int:
    return int(load_library().sasq_absmax_scale_workspace(int(numel)))


def sasq_absmax_scale(x, scale_out, workspace, bits: int = 8, stream=None) -> None:
    """scale_out[0] = max|x| / Qp (Eq. 1) of one calibration batch."""
    _dev(x, "x"); _dev(scale_out, "scale_out", torch.float32); _dev(workspace, "workspace")
    _check(load_library().sasq_absmax_scale(_ptr(x), x.numel(), _dt(x), int(bits), _ptr(scale_out), _ptr(workspace),
                                            _nbytes(workspace), _stream(stream)), "sasq_absmax_scale")


def sasq_quantize_weight(w, w_int, w_scale, bits: int = 8, stream=None) -> None:
    """w [N, K] fp32 -> w_int [N, K] int8 and w_scale [N] fp32, one factor per output channel."""
    _dev(w, "w", torch.float32); _dev(w_int, "w_int", torch.int8); _dev(w_scale, "w_scale", torch.float32)
    if w.dim() != 2 or tuple(w_int.shape) != tuple(w.shape) or w_scale.numel() != w.shape[0]:
        raise ValueError("w and w_int must be [N, K], w_scale [N]")
    _check(load_library().sasq_quantize_weight(_ptr(w), _ptr(w_int), _ptr(w_scale), w.shape[0], w.shape[1], int(bits),
                                               _stream(stream)), "sasq_quantize_weight")


def sasq_fakequant_fwd_bwd_static(x, grad_y, y, grad_x, grad_scale, scale, bits: int = 8, accumulate: bool = False,
                                  stream=None) -> None:
    """Fused forward + backward without any workspace argument: the reduction scratch is a fixed array inside the
    library, for callers that are not allowed to allocate (see include/sasq.h).  Calls on one device must not
    overlap; the first call on a device should be made outside stream capture."""
    _dev(x, "x"); _dev(grad_y, "grad_y", x.dtype); _dev(y, "y", x.dtype); _dev(grad_x, "grad_x", x.dtype)
    _dev(grad_scale, "grad_scale", torch.float32); _dev(scale, "scale", torch.float32)
    if grad_y.numel() != x.numel() or grad_x.numel() != x.numel() or y.numel() != x.numel():
        raise ValueError("grad_y, y and grad_x must have as many elements as x")
    _check(load_library().sasq_fakequant_fwd_bwd_static(_ptr(x), _ptr(grad_y), _ptr(y), _ptr(grad_x),
                                                        _ptr(grad_scale), int(bool(accumulate)), x.numel(), _dt(x),
                                                        _ptr(scale), int(bits), _stream(stream)),
           "sasq_fakequant_fwd_bwd_static")

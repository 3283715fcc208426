"""Python face of the SASQ CPU oracle (``sasq_oracle.cpp``).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH: only the test suite, the smoke check
and the benchmark's CPU-baseline leg may import this package.  It never imports
the CUDA package and shares nothing with it.

All 16-bit tensors cross this boundary as raw ``uint16`` bit patterns (numpy
arrays) together with a dtype tag: ``F16 = 0`` (IEEE binary16) or ``BF16 = 1``.
Helpers convert to and from torch CPU tensors by reinterpreting bits only.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

F16 = 0
BF16 = 1

FULL = 0        # quant, round, clamp, dequant (Sec. 4.2)
NO_ROUND = 1    # Table 3 "w/o round"
NO_CLAMP = 2    # Table 3 "w/o clamp"

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sasq_oracle.cpp")
_LIB = os.path.join(_HERE, "libsasq_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with contraction and fast-math off; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-fopenmp", "-ffp-contract=off", "-fno-fast-math",
               "-shared", "-fPIC", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.oracle_absmax_scale.restype = ctypes.c_float
        L.oracle_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().oracle_num_threads())


# ---------------------------------------------------------------------------
# marshalling helpers
# ---------------------------------------------------------------------------
def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def bits_of(t) -> tuple[np.ndarray, int]:
    """torch CPU fp16/bf16 tensor -> (uint16 bit array of the same shape, dtype tag)."""
    import torch
    assert t.device.type == "cpu"
    tag = {torch.float16: F16, torch.bfloat16: BF16}[t.dtype]
    return t.contiguous().view(torch.int16).numpy().view(np.uint16).copy(), tag


def tensor_of(bits: np.ndarray, tag: int):
    """uint16 bit array -> torch CPU tensor of the tagged dtype (bit reinterpretation)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16).copy())
    return t.view(torch.float16 if tag == F16 else torch.bfloat16)


def _i64(v):
    return ctypes.c_int64(int(v))


def _chk(rc):
    if rc != 0:
        raise ValueError("oracle rejected the arguments")


# ---------------------------------------------------------------------------
# the oracle's functions
# ---------------------------------------------------------------------------
def widen(bits: np.ndarray, tag: int) -> np.ndarray:
    bits = _u16(bits)
    out = np.empty(bits.shape, np.float32)
    lib().oracle_widen(_p(bits), _p(out), _i64(bits.size), ctypes.c_int(tag))
    return out


def narrow(vals: np.ndarray, tag: int) -> np.ndarray:
    vals = np.ascontiguousarray(vals, dtype=np.float32)
    out = np.empty(vals.shape, np.uint16)
    lib().oracle_narrow(_p(vals), _p(out), _i64(vals.size), ctypes.c_int(tag))
    return out


def absmax_scale(x: np.ndarray, tag: int, bits: int = 8) -> np.float32:
    """Eq. 1: S = max|X| / (2^(b-1) - 1)."""
    x = _u16(x)
    return np.float32(lib().oracle_absmax_scale(_p(x), _i64(x.size), ctypes.c_int(tag), ctypes.c_int(bits)))


def _rows_cols(x: np.ndarray):
    if x.ndim == 2:
        return x.shape
    return (1, x.size) if x.size else (0, 0)


def fakequant_fwd(x: np.ndarray, tag: int, s: float, bits: int = 8, variant: int = FULL, want_codes: bool = True):
    """Returns (y bits, codes int32 or None)."""
    x = _u16(x)
    rows, cols = _rows_cols(x)
    y = np.empty(x.shape, np.uint16)
    codes = np.empty(x.shape, np.int32) if (want_codes and variant != NO_ROUND) else None
    _chk(lib().oracle_fakequant_fwd(_p(x), _p(y), _p(codes), _i64(rows), _i64(cols), ctypes.c_int(tag),
                                    ctypes.c_float(s), ctypes.c_int(bits), ctypes.c_int(variant)))
    return y, codes


def fakequant_bwd(x: np.ndarray, g: np.ndarray, tag: int, s: float, bits: int = 8, variant: int = FULL):
    """Returns (dx bits, ds as python float holding the double sum)."""
    x = _u16(x)
    g = _u16(g)
    assert x.shape == g.shape
    rows, cols = _rows_cols(x)
    dx = np.empty(x.shape, np.uint16)
    ds = ctypes.c_double(0.0)
    _chk(lib().oracle_fakequant_bwd(_p(x), _p(g), _p(dx), ctypes.byref(ds), _i64(rows), _i64(cols),
                                    ctypes.c_int(tag), ctypes.c_float(s), ctypes.c_int(bits), ctypes.c_int(variant)))
    return dx, float(ds.value)


def fakequant_fwd_per_channel(x: np.ndarray, tag: int, s: np.ndarray, bits: int = 8):
    x = _u16(x)
    rows, cols = x.shape
    s = np.ascontiguousarray(s, dtype=np.float32)
    assert s.shape == (cols,)
    y = np.empty(x.shape, np.uint16)
    codes = np.empty(x.shape, np.int32)
    _chk(lib().oracle_fakequant_fwd_per_channel(_p(x), _p(y), _p(codes), _i64(rows), _i64(cols), ctypes.c_int(tag),
                                                _p(s), ctypes.c_int(bits)))
    return y, codes


def fakequant_bwd_per_channel(x: np.ndarray, g: np.ndarray, tag: int, s: np.ndarray, bits: int = 8):
    x = _u16(x)
    g = _u16(g)
    rows, cols = x.shape
    s = np.ascontiguousarray(s, dtype=np.float32)
    dx = np.empty(x.shape, np.uint16)
    ds = np.zeros((cols,), np.float64)
    _chk(lib().oracle_fakequant_bwd_per_channel(_p(x), _p(g), _p(dx), _p(ds), _i64(rows), _i64(cols),
                                                ctypes.c_int(tag), _p(s), ctypes.c_int(bits)))
    return dx, ds


def quantize_act(x: np.ndarray, tag: int, s: float, bits: int = 8) -> np.ndarray:
    x = _u16(x)
    rows, cols = _rows_cols(x)
    codes = np.empty(x.shape, np.int8)
    _chk(lib().oracle_quantize_act(_p(x), _p(codes), _i64(rows), _i64(cols), ctypes.c_int(tag), ctypes.c_float(s),
                                   ctypes.c_int(bits)))
    return codes


def quantize_weight(w: np.ndarray, bits: int = 8):
    """fp32 w[N, K] -> (int8 w_int[N, K], fp32 w_scale[N]); one factor per output channel."""
    w = np.ascontiguousarray(w, dtype=np.float32)
    N, K = w.shape
    w_int = np.empty((N, K), np.int8)
    w_scale = np.empty((N,), np.float32)
    _chk(lib().oracle_quantize_weight(_p(w), _p(w_int), _p(w_scale), _i64(N), _i64(K), ctypes.c_int(bits)))
    return w_int, w_scale


def int_gemm(x_int: np.ndarray, w_int: np.ndarray, row_begin: int = 0, row_end: int | None = None) -> np.ndarray:
    """acc[T, N] int32; rows outside [row_begin, row_end) are left zero."""
    x_int = np.ascontiguousarray(x_int, dtype=np.int8)
    w_int = np.ascontiguousarray(w_int, dtype=np.int8)
    T, K = x_int.shape
    N, K2 = w_int.shape
    assert K == K2
    row_end = T if row_end is None else row_end
    acc = np.zeros((T, N), np.int32)
    _chk(lib().oracle_int_gemm(_p(x_int), _p(w_int), _p(acc), _i64(T), _i64(N), _i64(K), _i64(row_begin),
                               _i64(row_end)))
    return acc


def int_gemm_i64(x_int: np.ndarray, w_int: np.ndarray) -> np.ndarray:
    x_int = np.ascontiguousarray(x_int, dtype=np.int8)
    w_int = np.ascontiguousarray(w_int, dtype=np.int8)
    T, K = x_int.shape
    N, _ = w_int.shape
    acc = np.zeros((T, N), np.int64)
    _chk(lib().oracle_int_gemm_i64(_p(x_int), _p(w_int), _p(acc), _i64(T), _i64(N), _i64(K)))
    return acc


def dequant(acc: np.ndarray, w_scale: np.ndarray, s_x: float, tag: int, bias: np.ndarray | None = None,
            row_begin: int = 0, row_end: int | None = None):
    """Returns (y bits [T, N], y32 fp32 [T, N]); rows outside the range are zero."""
    acc = np.ascontiguousarray(acc, dtype=np.int32)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    T, N = acc.shape
    row_end = T if row_end is None else row_end
    y = np.zeros((T, N), np.uint16)
    y32 = np.zeros((T, N), np.float32)
    b = None if bias is None else _u16(bias)
    _chk(lib().oracle_dequant(_p(acc), _p(w_scale), ctypes.c_float(s_x), _p(b), _p(y), _p(y32), _i64(T), _i64(N),
                              ctypes.c_int(tag), _i64(row_begin), _i64(row_end)))
    return y, y32


def w8a8_linear(x: np.ndarray, tag: int, w_int: np.ndarray, w_scale: np.ndarray, s_x: float, bits: int = 8,
                bias: np.ndarray | None = None, row_begin: int = 0, row_end: int | None = None):
    """Static W8A8 linear. Returns (y bits, y32, acc int32), rows outside the range zero."""
    x = _u16(x)
    w_int = np.ascontiguousarray(w_int, dtype=np.int8)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    T, K = x.shape
    N, K2 = w_int.shape
    assert K == K2 and w_scale.shape == (N,)
    row_end = T if row_end is None else row_end
    y = np.zeros((T, N), np.uint16)
    y32 = np.zeros((T, N), np.float32)
    acc = np.zeros((T, N), np.int32)
    scratch = np.zeros((T, K), np.int8)
    b = None if bias is None else _u16(bias)
    _chk(lib().oracle_w8a8_linear(_p(x), _p(w_int), _p(w_scale), ctypes.c_float(s_x), _p(b), _p(y), _p(y32), _p(acc),
                                  _p(scratch), _i64(T), _i64(N), _i64(K), ctypes.c_int(tag), ctypes.c_int(bits),
                                  _i64(row_begin), _i64(row_end)))
    return y, y32, acc


def w8a8_linear_grouped(x: np.ndarray, tag: int, w_int: np.ndarray, w_scale: np.ndarray, s_group: np.ndarray,
                        group: int, bits: int = 8, bias: np.ndarray | None = None):
    """Eq. 3: K cut into groups of `group` columns, one activation factor per group."""
    x = _u16(x)
    w_int = np.ascontiguousarray(w_int, dtype=np.int8)
    w_scale = np.ascontiguousarray(w_scale, dtype=np.float32)
    s_group = np.ascontiguousarray(s_group, dtype=np.float32)
    T, K = x.shape
    N, _ = w_int.shape
    y = np.zeros((T, N), np.uint16)
    y32 = np.zeros((T, N), np.float32)
    b = None if bias is None else _u16(bias)
    _chk(lib().oracle_w8a8_linear_grouped(_p(x), _p(w_int), _p(w_scale), _p(s_group), _i64(group), _p(b), _p(y),
                                          _p(y32), _i64(T), _i64(N), _i64(K), ctypes.c_int(tag), ctypes.c_int(bits)))
    return y, y32


def adamw_step(s, g, m, v, step: int, lr: float = 2e-4, beta1: float = 0.9, beta2: float = 0.999, eps: float = 1e-8,
               weight_decay: float = 0.01):
    """One AdamW step on the factors (Sec. 5.1: AdamW, lr 2e-4; the factors are the only trainable parameters,
    Sec. 4.2), written out in float64 with decoupled weight decay.  Returns the new (s, m, v); inputs untouched."""
    s = np.asarray(s, np.float64)
    g = np.asarray(g, np.float64)
    m = beta1 * np.asarray(m, np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, np.float64) + (1.0 - beta2) * g * g
    m_hat = m / (1.0 - beta1 ** step)
    v_hat = v / (1.0 - beta2 ** step)
    s_new = s - lr * (m_hat / (np.sqrt(v_hat) + eps) + weight_decay * s)
    return s_new, m, v


def w8a8_linear_dynamic(x: np.ndarray, tag: int, w_int: np.ndarray, w_scale: np.ndarray, bits: int = 8,
                        bias: np.ndarray | None = None):
    """Dynamic per-token W8A8 linear (Sec. 4.4, generation phase): every row is a tensor of its own with the
    max-based factor of Eq. 1 (an all-zero row takes factor 1), then Eq. 2.  Written as the per-tensor routines
    applied row by row.  Returns (y bits, acc int32, row factors fp32)."""
    x = _u16(x)
    T, K = x.shape
    N = w_int.shape[0]
    y = np.zeros((T, N), np.uint16)
    acc = np.zeros((T, N), np.int32)
    s_rows = np.zeros(T, np.float32)
    for t in range(T):
        row = x[t:t + 1]
        s = absmax_scale(row, tag, bits)
        if not s > 0:
            s = np.float32(1.0)
        s_rows[t] = s
        y_t, _, acc_t = w8a8_linear(row, tag, w_int, w_scale, float(s), bits, bias)
        y[t], acc[t] = y_t[0], acc_t[0]
    return y, acc, s_rows


def w8a8_linear_per_channel(x: np.ndarray, tag: int, w_int: np.ndarray, w_scale: np.ndarray, s_vec: np.ndarray,
                            bits: int = 8, bias: np.ndarray | None = None):
    """Static W8A8 linear with one activation factor per channel whose values were folded into the weights ahead of
    time (w_int, w_scale quantize w_fp[n,k] * s_vec[k]): Eq. 1 per channel, the integer GEMM, then Eq. 2 with the
    activation factor already inside the weights (output factor w_scale[n] alone).  Built from the pinned pieces.
    Returns (y bits, acc int32)."""
    _, codes = fakequant_fwd_per_channel(x, tag, s_vec, bits)
    acc = int_gemm(codes.astype(np.int8), w_int)
    y, _ = dequant(acc, w_scale, 1.0, tag, bias)
    return y, acc


def fp_weights_linear(x: np.ndarray, tag: int, w: np.ndarray, s: float, bits: int = 8, bias: np.ndarray | None = None):
    """Table 3's "FP weights" form (Eq. 5 and 6: quantization as a transform of the activations alone):
    Y = g(X) W^T with X' = g(X) the fake-quantized activations (the pinned forward) and the weights left in their
    16-bit floating-point type.  The contraction is a library matmul in float64; returns the float64 result before
    any narrowing, and sum_k |x'[t,k] w[n,k]| for error bounds."""
    xq, _ = fakequant_fwd(x, tag, s, bits, want_codes=False)
    a = widen(xq, tag).astype(np.float64)
    b = widen(_u16(w), tag).astype(np.float64)
    y = a @ b.T
    mag = np.abs(a) @ np.abs(b).T
    if bias is not None:
        bv = widen(_u16(bias), tag).astype(np.float64)
        y = y + bv[None, :]
        mag = mag + np.abs(bv)[None, :]
    return y, mag

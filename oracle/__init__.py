"""fp64 CPU oracle for RMSNorm / LayerNorm / softmax / cross-entropy forward and row-sum (ctypes wrapper).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import this package.  It shares nothing with the
CUDA library and never imports it.  All arithmetic lives in ``ak_oracle.c`` (plain C,
double precision, the textbook definition of each op); this file only marshals numpy
arrays.  Inputs are bf16 *bit patterns* (``uint16``); outputs are ``float64``.

Ops follow Table 3 of the paper (softmax / rmsnorm / layernorm / cross_ent / reduce rows) with the
semantics of the PyTorch reference implementation the paper names as its correctness
oracle (Section 6).  Readings the paper does not pin ("parity unpinned", PyTorch
convention): fully -inf softmax row -> NaN; inf/NaN inputs propagate; eps = 0 with a
zero row -> NaN; inf/NaN in a LayerNorm row -> NaN row; all rows ignored -> mean NaN; out-of-range target -> NaN row.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np

from .build import build as _build, LIB_PATH as _LIB_PATH

_lib = None


def _load():
    global _lib
    if _lib is None:
        _build()  # no-op when the shared object is newer than its source
        lib = ctypes.CDLL(_LIB_PATH)
        i64, f32 = ctypes.c_int64, ctypes.c_float
        p = ctypes.c_void_p
        lib.oracle_bf16_to_f64.argtypes = [p, p, i64]
        lib.oracle_bf16_to_f64.restype = None
        lib.oracle_set_threads.argtypes = [ctypes.c_int]
        lib.oracle_set_threads.restype = ctypes.c_int
        lib.oracle_f16_to_f64.argtypes = [p, p, i64]
        lib.oracle_f16_to_f64.restype = None
        lib.oracle_rmsnorm_dt.argtypes = [p, p, p, i64, i64, f32, ctypes.c_int]
        lib.oracle_rmsnorm_dt.restype = None
        lib.oracle_softmax_dt.argtypes = [p, p, i64, i64, ctypes.c_int]
        lib.oracle_softmax_dt.restype = None
        lib.oracle_xent_dt.argtypes = [p, p, i64, p, p, p, i64, i64, ctypes.c_int]
        lib.oracle_xent_dt.restype = None
        lib.oracle_layernorm_dt.argtypes = [p, p, p, p, i64, i64, f32, ctypes.c_int]
        lib.oracle_layernorm_dt.restype = None
        lib.oracle_rowsum_dt.argtypes = [p, p, i64, i64, ctypes.c_int]
        lib.oracle_rowsum_dt.restype = None
        lib.oracle_rope.argtypes = [p, p, i64, i64, i64, f32, i64, ctypes.c_int]
        lib.oracle_rope.restype = None
        lib.oracle_rmsnorm.argtypes = [p, p, p, i64, i64, f32]
        lib.oracle_rmsnorm.restype = None
        lib.oracle_layernorm.argtypes = [p, p, p, p, i64, i64, f32]
        lib.oracle_layernorm.restype = None
        lib.oracle_rowsum.argtypes = [p, p, i64, i64]
        lib.oracle_rowsum.restype = None
        lib.oracle_softmax.argtypes = [p, p, i64, i64]
        lib.oracle_softmax.restype = None
        lib.oracle_xent.argtypes = [p, p, i64, p, p, p, i64, i64]
        lib.oracle_xent.restype = None
        _lib = lib
    return _lib


def _bits(a, shape=None) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError(f"bf16 bit patterns must be uint16, got {a.dtype}")
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


DTYPES = {"bf16": 0, "f16": 1, "f32": 2}


def _elems(a, dtype: str, shape=None) -> np.ndarray:
    """Input array of element type ``dtype``: uint16 bit patterns for bf16 / f16, float32 for f32."""
    a = np.ascontiguousarray(a)
    want = np.float32 if dtype == "f32" else np.uint16
    if a.dtype != want:
        raise TypeError(f"{dtype} inputs must be {np.dtype(want)}, got {a.dtype}")
    if shape is not None and a.shape != shape:
        raise ValueError(f"expected shape {shape}, got {a.shape}")
    return a


def set_threads(n: int = 0) -> int:
    """Set (n > 0) or query (n = 0) the number of row-loop threads."""
    return int(_load().oracle_set_threads(int(n)))


def bf16_to_f64(bits) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    b = _bits(bits)
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_bf16_to_f64(b.ctypes.data, out.ctypes.data, b.size)
    return out


def f16_to_f64(bits) -> np.ndarray:
    """Exact widening of IEEE binary16 bit patterns to float64."""
    b = _bits(bits)
    out = np.empty(b.shape, dtype=np.float64)
    _load().oracle_f16_to_f64(b.ctypes.data, out.ctypes.data, b.size)
    return out


def rmsnorm_dt(x, w, eps: float, dtype: str) -> np.ndarray:
    """RMSNorm on inputs of element type ``dtype`` ("bf16", "f16": uint16 bits; "f32": float32)."""
    x = _elems(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    w = _elems(w, dtype, (D,))
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_rmsnorm_dt(x.ctypes.data, w.ctypes.data, y.ctypes.data, rows, D,
                              float(np.float32(eps)), DTYPES[dtype])
    return y


def softmax_dt(x, dtype: str) -> np.ndarray:
    x = _elems(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_softmax_dt(x.ctypes.data, y.ctypes.data, rows, D, DTYPES[dtype])
    return y


def xent_dt(logits, targets, dtype: str, ignore_index: int = -100):
    """Returns (loss_rows float64 [rows], loss_mean float, n_counted int)."""
    x = _elems(logits, dtype)
    if x.ndim != 2:
        raise ValueError("logits must be [rows, V]")
    rows, V = x.shape
    t = np.ascontiguousarray(targets)
    if t.dtype != np.int64 or t.shape != (rows,):
        raise TypeError("targets must be int64 [rows]")
    loss = np.empty((rows,), dtype=np.float64)
    mean = ctypes.c_double(float("nan"))
    cnt = ctypes.c_int64(0)
    _load().oracle_xent_dt(x.ctypes.data, t.ctypes.data, int(ignore_index), loss.ctypes.data,
                           ctypes.addressof(mean), ctypes.addressof(cnt), rows, V, DTYPES[dtype])
    return loss, float(mean.value), int(cnt.value)


def layernorm_dt(x, gamma, beta, eps: float, dtype: str) -> np.ndarray:
    """LayerNorm on inputs of element type ``dtype`` (see :func:`layernorm`)."""
    x = _elems(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    g = _elems(gamma, dtype, (D,))
    b = _elems(beta, dtype, (D,))
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_layernorm_dt(x.ctypes.data, g.ctypes.data, b.ctypes.data, y.ctypes.data, rows, D,
                                float(np.float32(eps)), DTYPES[dtype])
    return y


def rowsum_dt(x, dtype: str) -> np.ndarray:
    """out[r] = sum_j x[r, j] for inputs of element type ``dtype``, in float64."""
    x = _elems(x, dtype)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    out = np.empty((rows,), dtype=np.float64)
    _load().oracle_rowsum_dt(x.ctypes.data, out.ctypes.data, rows, D, DTYPES[dtype])
    return out


def rope(x, dtype: str, base: float = 10000.0, pos_offset: int = 0) -> np.ndarray:
    """Interleaved rotary embedding of x [n_seq, S, Dh] (element type ``dtype``): the pair
    (2i, 2i+1) at sequence index s is rotated by (pos_offset + s) * base^(-2i/Dh).  float64 out;
    ``base`` is first rounded to float32."""
    x = _elems(x, dtype)
    if x.ndim != 3 or x.shape[2] % 2:
        raise ValueError("x must be [n_seq, S, Dh] with even Dh")
    n_seq, S, Dh = x.shape
    y = np.empty((n_seq, S, Dh), dtype=np.float64)
    _load().oracle_rope(x.ctypes.data, y.ctypes.data, n_seq, S, Dh, float(np.float32(base)),
                        int(pos_offset), DTYPES[dtype])
    return y


def rmsnorm(x_bits, w_bits, eps: float) -> np.ndarray:
    """y[r, j] = x[r, j] * w[j] / sqrt(mean_j(x[r, :]^2) + eps), in float64.

    ``eps`` is first rounded to float32 (that is what the GPU entry point receives).
    """
    x = _bits(x_bits)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    w = _bits(w_bits, (D,))
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_rmsnorm(x.ctypes.data, w.ctypes.data, y.ctypes.data, rows, D,
                           float(np.float32(eps)))
    return y


def layernorm(x_bits, gamma_bits, beta_bits, eps: float) -> np.ndarray:
    """y[r, j] = (x[r, j] - mean_r) / sqrt(var_r + eps) * gamma[j] + beta[j] (biased variance),
    in float64; ``eps`` is first rounded to float32."""
    x = _bits(x_bits)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    g = _bits(gamma_bits, (D,))
    b = _bits(beta_bits, (D,))
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_layernorm(x.ctypes.data, g.ctypes.data, b.ctypes.data, y.ctypes.data, rows, D,
                             float(np.float32(eps)))
    return y


def rowsum(x_bits) -> np.ndarray:
    """out[r] = sum_j x[r, j], in float64."""
    x = _bits(x_bits)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    out = np.empty((rows,), dtype=np.float64)
    _load().oracle_rowsum(x.ctypes.data, out.ctypes.data, rows, D)
    return out


def softmax(x_bits) -> np.ndarray:
    """Row-wise exp(x - max) / sum exp(x - max) over the last dim, in float64."""
    x = _bits(x_bits)
    if x.ndim != 2:
        raise ValueError("x must be [rows, D]")
    rows, D = x.shape
    y = np.empty((rows, D), dtype=np.float64)
    _load().oracle_softmax(x.ctypes.data, y.ctypes.data, rows, D)
    return y


def xent(logits_bits, targets, ignore_index: int = -100):
    """Returns (loss_rows float64 [rows], loss_mean float, n_counted int)."""
    x = _bits(logits_bits)
    if x.ndim != 2:
        raise ValueError("logits must be [rows, V]")
    rows, V = x.shape
    t = np.ascontiguousarray(targets)
    if t.dtype != np.int64 or t.shape != (rows,):
        raise TypeError("targets must be int64 [rows]")
    loss = np.empty((rows,), dtype=np.float64)
    mean = ctypes.c_double(float("nan"))
    cnt = ctypes.c_int64(0)
    _load().oracle_xent(x.ctypes.data, t.ctypes.data, int(ignore_index),
                        loss.ctypes.data, ctypes.addressof(mean), ctypes.addressof(cnt),
                        rows, V)
    return loss, float(mean.value), int(cnt.value)

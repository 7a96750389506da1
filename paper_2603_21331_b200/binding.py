"""ctypes binding of ``libak.so``: argument marshalling only.

Every op runs in the CUDA library; nothing here computes, and there is no CPU or PyTorch
fallback: if the shared object is missing or a call fails, an exception is raised.

Two layers, same names as the C ABI (``include/ak.h``):

* ``lib()`` returns the ``ctypes.CDLL`` with typed entry points (``lib().ak_rmsnorm_fwd``
  etc.), taking raw device pointers as integers.
* ``ak_rmsnorm_fwd / ak_softmax_fwd / ak_xent_fwd`` (and ``*_host``, ``*_dt``,
  ``ak_layernorm_fwd``, ``ak_rowsum_fwd``, ``ak_rope_fwd``, ``ak_xent_vp_*``) take torch tensors,
  check dtype / contiguity / device, and pass ``data_ptr()`` and the current CUDA stream.
  PyTorch is used for device memory and streams only.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libak.so")

AK_OK = 0
AK_PATH_AUTO, AK_PATH_WARP, AK_PATH_CTA, AK_PATH_GENERIC, AK_PATH_SMEM, AK_PATH_CLUSTER = 0, 1, 2, 3, 4, 5
AK_XENT_AUTO, AK_XENT_ROW, AK_XENT_SPLIT = 0, 1, 2
AK_DTYPE_BF16, AK_DTYPE_F16, AK_DTYPE_F32 = 0, 1, 2
_DTYPES = {torch.bfloat16: AK_DTYPE_BF16, torch.float16: AK_DTYPE_F16, torch.float32: AK_DTYPE_F32}

_i64, _f32, _int, _p, _sz = (ctypes.c_int64, ctypes.c_float, ctypes.c_int, ctypes.c_void_p,
                             ctypes.c_size_t)

# name -> (restype, argtypes); mirrors include/ak.h one to one
SIGNATURES = {
    "ak_rmsnorm_fwd": (_int, [_p, _p, _p, _i64, _i64, _f32, _p]),
    "ak_rmsnorm_fwd_path": (_int, [_p, _p, _p, _i64, _i64, _f32, _p, _int]),
    "ak_rmsnorm_fwd_dt": (_int, [_p, _p, _p, _i64, _i64, _f32, _int, _p, _int]),
    "ak_softmax_fwd_dt": (_int, [_p, _p, _i64, _i64, _int, _p, _int]),
    "ak_xent_fwd_dt": (_int, [_p, _p, _i64, _p, _p, _i64, _i64, _int, _p, _int, _int]),
    "ak_choose_path_dt": (_int, [_int, _i64, _i64, _int, _int]),
    "ak_layernorm_fwd_dt": (_int, [_p, _p, _p, _p, _i64, _i64, _f32, _int, _p, _int]),
    "ak_rowsum_fwd_dt": (_int, [_p, _p, _i64, _i64, _int, _p]),
    "ak_rope_fwd": (_int, [_p, _p, _i64, _i64, _i64, _f32, _i64, _int, _p]),
    "ak_xent_vp_nsplit": (_int, [_i64, _i64]),
    "ak_xent_vp_partial_bytes": (_sz, [_i64, _int]),
    "ak_xent_vp_partial": (_int, [_p, _p, _i64, _i64, _i64, _p, _i64, _i64, _int, _int, _p]),
    "ak_xent_vp_merge": (_int, [_p, _int, _int, _p, _i64, _i64, _p, _p, _i64, _p]),
    "ak_layernorm_fwd": (_int, [_p, _p, _p, _p, _i64, _i64, _f32, _p]),
    "ak_layernorm_fwd_path": (_int, [_p, _p, _p, _p, _i64, _i64, _f32, _p, _int]),
    "ak_rowsum_fwd": (_int, [_p, _p, _i64, _i64, _p]),
    "ak_softmax_fwd": (_int, [_p, _p, _i64, _i64, _p]),
    "ak_softmax_fwd_path": (_int, [_p, _p, _i64, _i64, _p, _int]),
    "ak_xent_fwd": (_int, [_p, _p, _i64, _p, _p, _i64, _i64, _p]),
    "ak_xent_workspace_bytes": (_sz, [_i64, _i64]),
    "ak_xent_fwd_ws": (_int, [_p, _p, _i64, _p, _p, _i64, _i64, _p, _sz, _p]),
    "ak_xent_fwd_path": (_int, [_p, _p, _i64, _p, _p, _i64, _i64, _p, _int, _int]),
    "ak_xent_fwd_static": (_int, [_p, _p, _i64, _p, _p, _i64, _i64, _p]),
    "ak_xent_sum_count": (_int, [_p, _p, _i64, _i64, _p, _p]),
    "ak_xent_mean_merge": (_int, [_p, _i64, _p, _p]),
    "ak_rmsnorm_fwd_host": (_int, [_p, _p, _p, _i64, _i64, _f32]),
    "ak_softmax_fwd_host": (_int, [_p, _p, _i64, _i64]),
    "ak_xent_fwd_host": (_int, [_p, _p, _i64, _p, _p, _i64, _i64]),
    "ak_host_arena_release": (_int, []),
    "ak_sol_copy": (_int, [_p, _p, _sz, _p]),
    "ak_sol_read": (_int, [_p, _sz, _p, _p]),
    "ak_rmsnorm_choose_path": (_int, [_i64, _i64, _int]),
    "ak_layernorm_choose_path": (_int, [_i64, _i64, _int]),
    "ak_softmax_choose_path": (_int, [_i64, _i64, _int]),
    "ak_xent_choose_path": (_int, [_i64, _i64, ctypes.POINTER(_int)]),
    "ak_launch_count": (_i64, []),
    "ak_sm_count": (_int, []),
    "ak_wait_timeouts": (_int, []),
    "ak_status_string": (ctypes.c_char_p, [_int]),
    "ak_version": (_int, []),
}

_lib = None


class AkError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        msg = lib().ak_status_string(status).decode()
        super().__init__(f"{where} failed: status {status} ({msg})")


def lib() -> ctypes.CDLL:
    """Load libak.so (once).  Raises if it has not been built: there is no fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} not found: build it with `python -m paper_2603_21331_b200.build` "
                "(the ops have no CPU or PyTorch fallback)")
        l = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(l, name)
            fn.restype = res
            fn.argtypes = args
        _lib = l
    return _lib


def _check(status: int, where: str) -> None:
    if status != AK_OK:
        raise AkError(status, where)


# the raw handle of the current stream without building a torch.cuda.Stream object (about 2 us
# less per call, which counts for decoding-sized launches); absent in some builds of torch
_raw_current_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream_ptr(stream, like: Optional[torch.Tensor] = None) -> int:
    if stream is None:
        if _raw_current_stream is not None and like is not None:
            return _raw_current_stream(like.device.index)
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, torch.cuda.Stream):
        return stream.cuda_stream
    return int(stream)


class _on_device_of:
    """Makes the tensors' device the current CUDA device around a library call (the library
    launches on the current device; function attributes, scratch pools and streams belong to
    it) and puts the previous one back.  Tensors on different devices are refused."""
    __slots__ = ("index", "previous")

    def __init__(self, *tensors):
        index = None
        for t in tensors:
            if t is None:
                continue
            if index is None:
                index = t.device.index
            elif t.device.index != index:
                raise ValueError("all tensors of a call must be on the same CUDA device")
        self.index = index
        self.previous = None

    def __enter__(self):
        if self.index is not None:
            current = torch.cuda.current_device()
            if current != self.index:
                self.previous = current
                torch.cuda.set_device(self.index)
        return self

    def __exit__(self, *exc):
        if self.previous is not None:
            torch.cuda.set_device(self.previous)
        return False


def _dev_bf16(t: torch.Tensor, name: str, ndim: int) -> None:
    if not (t.is_cuda and t.dtype == torch.bfloat16 and t.dim() == ndim and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA bfloat16 tensor with {ndim} dims")


def _host(t: torch.Tensor, name: str, dtype, ndim: int) -> None:
    if t.is_cuda or t.dtype != dtype or t.dim() != ndim or not t.is_contiguous():
        raise TypeError(f"{name} must be a contiguous CPU {dtype} tensor with {ndim} dims")


# ------------------------------------------------------------------------- device tensors
def ak_rmsnorm_fwd(x: torch.Tensor, w: torch.Tensor, y: Optional[torch.Tensor] = None,
                   eps: float = 1e-6, stream=None, path: int = AK_PATH_AUTO) -> torch.Tensor:
    _dev_bf16(x, "x", 2)
    _dev_bf16(w, "w", 1)
    rows, D = x.shape
    if w.shape[0] != D:
        raise ValueError("w must have D elements")
    if y is None:
        y = torch.empty_like(x)
    _dev_bf16(y, "y", 2)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, w, y):
        _check(lib().ak_rmsnorm_fwd_path(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, D, eps,
                                         _stream_ptr(stream, x), path), "ak_rmsnorm_fwd")
    return y


def _dev_dt(t: torch.Tensor, name: str, ndim: int, dtype=None) -> int:
    want = t.dtype if dtype is None else dtype
    if want not in _DTYPES or not (t.is_cuda and t.dtype == want and t.dim() == ndim and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA bf16 / fp16 / fp32 tensor with {ndim} dims"
                        + ("" if dtype is None else f" of dtype {dtype}"))
    return _DTYPES[want]


def ak_rmsnorm_fwd_dt(x: torch.Tensor, w: torch.Tensor, y: Optional[torch.Tensor] = None,
                      eps: float = 1e-6, stream=None, path: int = AK_PATH_AUTO) -> torch.Tensor:
    """RMSNorm in the element type of x (bf16, fp16 or fp32); w and y share it."""
    dt = _dev_dt(x, "x", 2)
    _dev_dt(w, "w", 1, x.dtype)
    rows, D = x.shape
    if w.shape[0] != D:
        raise ValueError("w must have D elements")
    if y is None:
        y = torch.empty_like(x)
    _dev_dt(y, "y", 2, x.dtype)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, w, y):
        _check(lib().ak_rmsnorm_fwd_dt(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, D, eps, dt,
                                       _stream_ptr(stream, x), path), "ak_rmsnorm_fwd_dt")
    return y


def ak_softmax_fwd_dt(x: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None,
                      path: int = AK_PATH_AUTO) -> torch.Tensor:
    """Softmax over the last dim in the element type of x (bf16, fp16 or fp32)."""
    dt = _dev_dt(x, "x", 2)
    rows, D = x.shape
    if y is None:
        y = torch.empty_like(x)
    _dev_dt(y, "y", 2, x.dtype)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, y):
        _check(lib().ak_softmax_fwd_dt(x.data_ptr(), y.data_ptr(), rows, D, dt, _stream_ptr(stream, x), path),
               "ak_softmax_fwd_dt")
    return y


def ak_xent_fwd_dt(logits: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                   stream=None, path: int = AK_XENT_AUTO, nsplit: int = 0,
                   want_mean: bool = True) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """Cross-entropy on logits of type bf16, fp16 or fp32; losses are fp32."""
    dt = _dev_dt(logits, "logits", 2)
    rows, V = logits.shape
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.shape == (rows,)
            and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    loss_rows = torch.empty((rows,), dtype=torch.float32, device=logits.device)
    loss_mean = torch.empty((1,), dtype=torch.float32, device=logits.device) if want_mean else None
    with _on_device_of(logits, targets, loss_rows, loss_mean):
        _check(lib().ak_xent_fwd_dt(logits.data_ptr(), targets.data_ptr(), ignore_index, loss_rows.data_ptr(),
                                    loss_mean.data_ptr() if want_mean else None, rows, V, dt,
                                    _stream_ptr(stream, logits), path, nsplit), "ak_xent_fwd_dt")
    return loss_rows, loss_mean


def ak_layernorm_fwd_dt(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor,
                        y: Optional[torch.Tensor] = None, eps: float = 1e-5, stream=None,
                        path: int = AK_PATH_AUTO) -> torch.Tensor:
    """LayerNorm in the element type of x (bf16, fp16 or fp32); gamma, beta and y share it."""
    dt = _dev_dt(x, "x", 2)
    _dev_dt(gamma, "gamma", 1, x.dtype)
    _dev_dt(beta, "beta", 1, x.dtype)
    rows, D = x.shape
    if gamma.shape[0] != D or beta.shape[0] != D:
        raise ValueError("gamma and beta must have D elements")
    if y is None:
        y = torch.empty_like(x)
    _dev_dt(y, "y", 2, x.dtype)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, gamma, beta, y):
        _check(lib().ak_layernorm_fwd_dt(x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), y.data_ptr(), rows, D,
                                         eps, dt, _stream_ptr(stream, x), path), "ak_layernorm_fwd_dt")
    return y


def ak_rowsum_fwd_dt(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Row sums (fp32) of x in bf16, fp16 or fp32."""
    dt = _dev_dt(x, "x", 2)
    rows, D = x.shape
    if out is None:
        out = torch.empty((rows,), dtype=torch.float32, device=x.device)
    if not (out.is_cuda and out.dtype == torch.float32 and out.shape == (rows,) and out.is_contiguous()):
        raise TypeError("out must be a contiguous CUDA float32 tensor [rows]")
    with _on_device_of(x, out):
        _check(lib().ak_rowsum_fwd_dt(x.data_ptr(), out.data_ptr(), rows, D, dt, _stream_ptr(stream, x)),
               "ak_rowsum_fwd_dt")
    return out


def ak_rope_fwd(x: torch.Tensor, y: Optional[torch.Tensor] = None, base: float = 10000.0,
                pos_offset: int = 0, stream=None) -> torch.Tensor:
    """Interleaved rotary embedding of x [n_seq, S, Dh] (bf16, fp16 or fp32); y may be x."""
    dt = _dev_dt(x, "x", 3)
    n_seq, S, Dh = x.shape
    if y is None:
        y = torch.empty_like(x)
    _dev_dt(y, "y", 3, x.dtype)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, y):
        _check(lib().ak_rope_fwd(x.data_ptr(), y.data_ptr(), n_seq, S, Dh, base, pos_offset, dt,
                                 _stream_ptr(stream, x)), "ak_rope_fwd")
    return y


def ak_xent_vp_nsplit(rows: int, V_local: int) -> int:
    return int(lib().ak_xent_vp_nsplit(rows, V_local))


def ak_xent_vp_partial(logits_shard: torch.Tensor, targets: torch.Tensor, vocab_start: int, V_total: int,
                       nsplit: int = 0, ignore_index: int = -100, partial: Optional[torch.Tensor] = None,
                       stream=None) -> torch.Tensor:
    """Phase 1 of the vocabulary-parallel cross-entropy on this rank's [rows, V_local] shard.
    Returns the partial buffer: float32 [rows, nsplit + 1, 2]."""
    dt = _dev_dt(logits_shard, "logits_shard", 2)
    rows, V_local = logits_shard.shape
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.shape == (rows,)
            and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    if nsplit == 0:
        nsplit = ak_xent_vp_nsplit(rows, V_local)
    if partial is None:
        # zero-filled so that the entries of unread rows are defined bytes for the exchange
        partial = torch.zeros((rows, nsplit + 1, 2), dtype=torch.float32, device=logits_shard.device)
    if not (partial.is_cuda and partial.dtype == torch.float32 and partial.shape == (rows, nsplit + 1, 2)
            and partial.is_contiguous()):
        raise TypeError("partial must be a contiguous CUDA float32 tensor [rows, nsplit + 1, 2]")
    with _on_device_of(logits_shard, targets, partial):
        _check(lib().ak_xent_vp_partial(logits_shard.data_ptr(), targets.data_ptr(), ignore_index, vocab_start,
                                        V_total, partial.data_ptr(), rows, V_local, nsplit, dt,
                                        _stream_ptr(stream, logits_shard)), "ak_xent_vp_partial")
    return partial


def ak_xent_vp_merge(partials: torch.Tensor, targets: torch.Tensor, V_total: int, ignore_index: int = -100,
                     want_mean: bool = True, stream=None) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    """Phase 2: ``partials`` = float32 [nranks, rows, nsplit + 1, 2] (all ranks' buffers in rank
    order).  Returns (loss_rows fp32 [rows], loss_mean fp32 [1] or None)."""
    if not (partials.is_cuda and partials.dtype == torch.float32 and partials.dim() == 4
            and partials.shape[3] == 2 and partials.is_contiguous()):
        raise TypeError("partials must be a contiguous CUDA float32 tensor [nranks, rows, nsplit + 1, 2]")
    nranks, rows, ns1, _ = partials.shape
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.shape == (rows,)
            and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    loss_rows = torch.empty((rows,), dtype=torch.float32, device=partials.device)
    loss_mean = torch.empty((1,), dtype=torch.float32, device=partials.device) if want_mean else None
    with _on_device_of(partials, targets, loss_rows, loss_mean):
        _check(lib().ak_xent_vp_merge(partials.data_ptr(), nranks, ns1 - 1, targets.data_ptr(), ignore_index,
                                      V_total, loss_rows.data_ptr(), loss_mean.data_ptr() if want_mean else None,
                                      rows, _stream_ptr(stream, partials)), "ak_xent_vp_merge")
    return loss_rows, loss_mean


def ak_choose_path_dt(op: str, rows: int, D: int, dtype: torch.dtype, aligned16: bool = True) -> int:
    return int(lib().ak_choose_path_dt({"rmsnorm": 0, "softmax": 1, "layernorm": 2}[op], rows, D, int(aligned16), _DTYPES[dtype]))


def ak_layernorm_fwd(x: torch.Tensor, gamma: torch.Tensor, beta: torch.Tensor,
                     y: Optional[torch.Tensor] = None, eps: float = 1e-5, stream=None,
                     path: int = AK_PATH_AUTO) -> torch.Tensor:
    _dev_bf16(x, "x", 2)
    _dev_bf16(gamma, "gamma", 1)
    _dev_bf16(beta, "beta", 1)
    rows, D = x.shape
    if gamma.shape[0] != D or beta.shape[0] != D:
        raise ValueError("gamma and beta must have D elements")
    if y is None:
        y = torch.empty_like(x)
    _dev_bf16(y, "y", 2)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, gamma, beta, y):
        _check(lib().ak_layernorm_fwd_path(x.data_ptr(), gamma.data_ptr(), beta.data_ptr(), y.data_ptr(),
                                           rows, D, eps, _stream_ptr(stream, x), path), "ak_layernorm_fwd")
    return y


def ak_rowsum_fwd(x: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    _dev_bf16(x, "x", 2)
    rows, D = x.shape
    if out is None:
        out = torch.empty((rows,), dtype=torch.float32, device=x.device)
    if not (out.is_cuda and out.dtype == torch.float32 and out.shape == (rows,) and out.is_contiguous()):
        raise TypeError("out must be a contiguous CUDA float32 tensor [rows]")
    with _on_device_of(x, out):
        _check(lib().ak_rowsum_fwd(x.data_ptr(), out.data_ptr(), rows, D, _stream_ptr(stream, x)), "ak_rowsum_fwd")
    return out


def ak_softmax_fwd(x: torch.Tensor, y: Optional[torch.Tensor] = None, stream=None,
                   path: int = AK_PATH_AUTO) -> torch.Tensor:
    _dev_bf16(x, "x", 2)
    rows, D = x.shape
    if y is None:
        y = torch.empty_like(x)
    _dev_bf16(y, "y", 2)
    if y.shape != x.shape:
        raise ValueError("y must have the shape of x")
    with _on_device_of(x, y):
        _check(lib().ak_softmax_fwd_path(x.data_ptr(), y.data_ptr(), rows, D, _stream_ptr(stream, x), path),
               "ak_softmax_fwd")
    return y


def ak_xent_fwd(logits: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                loss_rows: Optional[torch.Tensor] = None, loss_mean: Optional[torch.Tensor] = None,
                stream=None, path: int = AK_XENT_AUTO, nsplit: int = 0,
                want_mean: bool = True) -> Tuple[torch.Tensor, Optional[torch.Tensor]]:
    _dev_bf16(logits, "logits", 2)
    rows, V = logits.shape
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.shape == (rows,)
            and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    if loss_rows is None:
        loss_rows = torch.empty((rows,), dtype=torch.float32, device=logits.device)
    if loss_mean is None and want_mean:
        loss_mean = torch.empty((1,), dtype=torch.float32, device=logits.device)
    for t, n in ((loss_rows, rows), (loss_mean, 1)):
        if t is not None and not (t.is_cuda and t.dtype == torch.float32 and t.numel() == n
                                  and t.is_contiguous()):
            raise TypeError("loss buffers must be contiguous CUDA float32 tensors")
    mean_ptr = loss_mean.data_ptr() if loss_mean is not None else None
    with _on_device_of(logits, targets, loss_rows, loss_mean):
        _check(lib().ak_xent_fwd_path(logits.data_ptr(), targets.data_ptr(), ignore_index,
                                      loss_rows.data_ptr(), mean_ptr, rows, V, _stream_ptr(stream, logits),
                                      path, nsplit), "ak_xent_fwd")
    return loss_rows, loss_mean


def ak_xent_fwd_static(logits: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                       loss_rows: Optional[torch.Tensor] = None,
                       loss_mean: Optional[torch.Tensor] = None, stream=None):
    """Cross-entropy forward for callers that may not allocate device memory at call time
    (pre-sized arenas, hard GPU quotas, allocator-free hot loops): the library's own fixed
    1 MiB scratch is used, nothing is allocated by the call itself.  Pass ``loss_rows`` and
    ``loss_mean`` to keep this wrapper from creating them.  Raises AkError with status 7 when
    rows * nsplit * 8 bytes exceeds 1 MiB or rows > 65535.  Calls that overlap on the GPU
    share the scratch and race; the first call on a device should precede any stream capture."""
    _dev_bf16(logits, "logits", 2)
    rows, V = logits.shape
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.shape == (rows,)
            and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    if loss_rows is None:
        loss_rows = torch.empty((rows,), dtype=torch.float32, device=logits.device)
    if loss_mean is None:
        loss_mean = torch.empty((1,), dtype=torch.float32, device=logits.device)
    with _on_device_of(logits, targets, loss_rows, loss_mean):
        _check(lib().ak_xent_fwd_static(logits.data_ptr(), targets.data_ptr(), ignore_index,
                                        loss_rows.data_ptr(), loss_mean.data_ptr(), rows, V,
                                        _stream_ptr(stream, logits)), "ak_xent_fwd_static")
    return loss_rows, loss_mean


def ak_xent_sum_count(loss_rows: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                      out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """{fp64 sum of the counted rows' losses, their count} of this rank's block of rows -> float64 [2]
    (the 16 bytes a rank contributes to the mean over row shards)."""
    rows = loss_rows.numel()
    if not (loss_rows.is_cuda and loss_rows.dtype == torch.float32 and loss_rows.is_contiguous()):
        raise TypeError("loss_rows must be a contiguous CUDA float32 tensor")
    if not (targets.is_cuda and targets.dtype == torch.int64 and targets.numel() == rows and targets.is_contiguous()):
        raise TypeError("targets must be a contiguous CUDA int64 tensor [rows]")
    if out is None:
        out = torch.empty((2,), dtype=torch.float64, device=loss_rows.device)
    if not (out.is_cuda and out.dtype == torch.float64 and out.numel() == 2 and out.is_contiguous()):
        raise TypeError("out must be a contiguous CUDA float64 tensor with 2 elements")
    with _on_device_of(loss_rows, targets, out):
        _check(lib().ak_xent_sum_count(loss_rows.data_ptr() if rows else None, targets.data_ptr() if rows else None,
                                       ignore_index, rows, out.data_ptr(), _stream_ptr(stream, loss_rows)),
               "ak_xent_sum_count")
    return out


def ak_xent_mean_merge(pairs: torch.Tensor, out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """Mean over row shards: ``pairs`` = float64 [n, 2] of (sum, count) in rank order, added in
    that order -> float32 [1] (NaN when nothing counts)."""
    if not (pairs.is_cuda and pairs.dtype == torch.float64 and pairs.dim() == 2 and pairs.shape[1] == 2
            and pairs.is_contiguous()):
        raise TypeError("pairs must be a contiguous CUDA float64 tensor [n, 2]")
    if out is None:
        out = torch.empty((1,), dtype=torch.float32, device=pairs.device)
    if not (out.is_cuda and out.dtype == torch.float32 and out.numel() == 1):
        raise TypeError("out must be a CUDA float32 tensor with 1 element")
    with _on_device_of(pairs, out):
        _check(lib().ak_xent_mean_merge(pairs.data_ptr() if pairs.shape[0] else None, pairs.shape[0], out.data_ptr(),
                                        _stream_ptr(stream, pairs)),
               "ak_xent_mean_merge")
    return out


def ak_xent_workspace_bytes(rows: int, V: int) -> int:
    return int(lib().ak_xent_workspace_bytes(rows, V))


def ak_xent_fwd_ws(logits: torch.Tensor, targets: torch.Tensor, workspace: Optional[torch.Tensor],
                   ignore_index: int = -100, loss_rows: Optional[torch.Tensor] = None,
                   loss_mean: Optional[torch.Tensor] = None, stream=None):
    _dev_bf16(logits, "logits", 2)
    rows, V = logits.shape
    if loss_rows is None:
        loss_rows = torch.empty((rows,), dtype=torch.float32, device=logits.device)
    if loss_mean is None:
        loss_mean = torch.empty((1,), dtype=torch.float32, device=logits.device)
    ws_ptr = workspace.data_ptr() if workspace is not None else None
    ws_bytes = workspace.numel() * workspace.element_size() if workspace is not None else 0
    with _on_device_of(logits, targets, loss_rows, loss_mean, workspace):
        _check(lib().ak_xent_fwd_ws(logits.data_ptr(), targets.data_ptr(), ignore_index,
                                    loss_rows.data_ptr(), loss_mean.data_ptr(), rows, V, ws_ptr, ws_bytes,
                                    _stream_ptr(stream, logits)), "ak_xent_fwd_ws")
    return loss_rows, loss_mean


# ------------------------------------------------------------------------- host tensors
def ak_rmsnorm_fwd_host(x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, eps: float = 1e-6) -> torch.Tensor:
    _host(x, "x", torch.bfloat16, 2)
    _host(w, "w", torch.bfloat16, 1)
    _host(y, "y", torch.bfloat16, 2)
    rows, D = x.shape
    _check(lib().ak_rmsnorm_fwd_host(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, D, eps),
           "ak_rmsnorm_fwd_host")
    return y


def ak_softmax_fwd_host(x: torch.Tensor, y: torch.Tensor) -> torch.Tensor:
    _host(x, "x", torch.bfloat16, 2)
    _host(y, "y", torch.bfloat16, 2)
    rows, D = x.shape
    _check(lib().ak_softmax_fwd_host(x.data_ptr(), y.data_ptr(), rows, D), "ak_softmax_fwd_host")
    return y


def ak_xent_fwd_host(logits: torch.Tensor, targets: torch.Tensor, loss_rows: torch.Tensor,
                     loss_mean: Optional[torch.Tensor], ignore_index: int = -100):
    _host(logits, "logits", torch.bfloat16, 2)
    _host(targets, "targets", torch.int64, 1)
    _host(loss_rows, "loss_rows", torch.float32, 1)
    rows, V = logits.shape
    mean_ptr = loss_mean.data_ptr() if loss_mean is not None else None
    _check(lib().ak_xent_fwd_host(logits.data_ptr(), targets.data_ptr(), ignore_index,
                                  loss_rows.data_ptr(), mean_ptr, rows, V), "ak_xent_fwd_host")
    return loss_rows, loss_mean


# ------------------------------------------------------------------------- introspection
def ak_rmsnorm_choose_path(rows: int, D: int, aligned16: bool = True) -> int:
    return int(lib().ak_rmsnorm_choose_path(rows, D, int(aligned16)))


def ak_layernorm_choose_path(rows: int, D: int, aligned16: bool = True) -> int:
    return int(lib().ak_layernorm_choose_path(rows, D, int(aligned16)))


def ak_softmax_choose_path(rows: int, D: int, aligned16: bool = True) -> int:
    return int(lib().ak_softmax_choose_path(rows, D, int(aligned16)))


def ak_xent_choose_path(rows: int, V: int) -> Tuple[int, int]:
    ns = ctypes.c_int(0)
    path = int(lib().ak_xent_choose_path(rows, V, ctypes.byref(ns)))
    return path, int(ns.value)


def ak_sm_count() -> int:
    return int(lib().ak_sm_count())


def ak_wait_timeouts() -> int:
    """0 if no bounded wait of a kernel ever gave up on the current device (see ak.h); synchronises."""
    return int(lib().ak_wait_timeouts())


def ak_launch_count() -> int:
    return int(lib().ak_launch_count())


def ak_version() -> int:
    return int(lib().ak_version())


def ak_status_string(status: int) -> str:
    return lib().ak_status_string(status).decode()

"""Comparison rules shared by the GPU parity tests.

bf16 outputs: the GPU value (widened exactly) must satisfy
    |gpu - ref| <= 1.6e-2 * max(1, |ref|)          (two bf16 ulps, the benchmark's bar)
and where ref is NaN the GPU value must be NaN, where ref is +-inf it must be the same
infinity, where ref is finite it must be finite.  A tighter secondary bound (one
round-to-nearest-even step, 2^-8 relative, plus the fp32 evaluation error) is reported
and asserted for finite references as well.

fp32 losses: |gpu - ref| <= 1e-5 * max(1, |ref|).  (A strictly relative 1e-5 is not
attainable when the true loss is far below fp32 epsilon, e.g. log1p(V e^-30).)
"""
from __future__ import annotations

import numpy as np
import torch

BF16_TOL = 1.6e-2
BF16_TIGHT = 2.0 ** -8 * 1.02 + 2e-6   # one RNE rounding + fp32 arithmetic slack
LOSS_TOL = 1e-5


def bf16_tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    bits = t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def assert_bf16_close(gpu: torch.Tensor, ref: np.ndarray, what: str = "", tight: bool = True):
    got = bf16_tensor_to_f64(gpu).reshape(ref.shape)
    nan_ref = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan_ref), f"{what}: NaN pattern differs"
    inf_ref = np.isinf(ref)
    assert np.array_equal(np.isinf(got), inf_ref), f"{what}: inf pattern differs"
    assert np.array_equal(got[inf_ref], ref[inf_ref]), f"{what}: inf sign differs"
    fin = ~(nan_ref | inf_ref)
    err = np.abs(got[fin] - ref[fin])
    bound = BF16_TOL * np.maximum(1.0, np.abs(ref[fin]))
    worst = float(np.max(err / bound)) if err.size else 0.0
    assert worst <= 1.0, f"{what}: max err/bound = {worst:.3f}"
    if tight and err.size:
        # smallest positive bf16 normal is ~1.2e-38; below that outputs may flush to zero
        tb = BF16_TIGHT * np.abs(ref[fin]) + 1.2e-38
        worst_t = float(np.max(err / tb))
        assert worst_t <= 1.0, f"{what}: exceeds one-rounding bound by {worst_t:.3f}x"
    return worst


# fp16 / fp32 outputs (derived from the arithmetic, the benchmark's bar being stated for bf16
# only): main bound = two units in the last place of the type relative to max(1, |ref|) for
# fp16 (2 * 2^-11), 1e-5 for fp32 (fp32 accumulation, rsqrt / ex2 approximations of ~2^-22 and
# the rounding of x*log2e at |x - m| up to ~100); tight bound = one rounding to nearest plus
# the fp32 evaluation error, relative to |ref|, plus the type's subnormal quantum.
DT_TOL = {torch.float16: 1.0e-3, torch.float32: 1.0e-5}
DT_TIGHT = {torch.float16: (2.0 ** -11 * 1.02 + 4e-6, 2.0 ** -24), torch.float32: (1.0e-5, 1e-37)}


def assert_close_dt(gpu: torch.Tensor, ref: np.ndarray, what: str = "", tight: bool = True):
    """Element-wise comparison of a bf16 / fp16 / fp32 GPU output with the fp64 reference."""
    if gpu.dtype == torch.bfloat16:
        return assert_bf16_close(gpu, ref, what, tight)
    got = gpu.detach().cpu().double().numpy().reshape(ref.shape)
    nan_ref = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan_ref), f"{what}: NaN pattern differs"
    inf_ref = np.isinf(ref)
    assert np.array_equal(np.isinf(got), inf_ref), f"{what}: inf pattern differs"
    assert np.array_equal(got[inf_ref], ref[inf_ref]), f"{what}: inf sign differs"
    fin = ~(nan_ref | inf_ref)
    err = np.abs(got[fin] - ref[fin])
    bound = DT_TOL[gpu.dtype] * np.maximum(1.0, np.abs(ref[fin]))
    worst = float(np.max(err / bound)) if err.size else 0.0
    assert worst <= 1.0, f"{what}: max err/bound = {worst:.3f}"
    if tight and err.size:
        rel, quantum = DT_TIGHT[gpu.dtype]
        worst_t = float(np.max(err / (rel * np.abs(ref[fin]) + quantum)))
        assert worst_t <= 1.0, f"{what}: exceeds one-rounding bound by {worst_t:.3f}x"
    return worst


def assert_close_on_device(gpu: torch.Tensor, ref: np.ndarray, what: str = "", tight: bool = True):
    """The rules of assert_close_dt for whole benchmark-sized tensors: the fp64 reference is
    copied to the GPU tensor's device and the element-by-element comparison runs there in fp64
    (widening the output to fp64 is exact), so that every element of a 500 MB output can be
    checked in seconds.  Only the comparison runs on the device; the reference is the CPU checker's."""
    dev = gpu.device
    r = torch.from_numpy(np.ascontiguousarray(ref)).to(dev)
    g = gpu.detach().double().reshape(r.shape)
    nan_ref, inf_ref = torch.isnan(r), torch.isinf(r)
    assert torch.equal(torch.isnan(g), nan_ref), f"{what}: NaN pattern differs"
    assert torch.equal(torch.isinf(g), inf_ref), f"{what}: inf pattern differs"
    assert torch.equal(g[inf_ref], r[inf_ref]), f"{what}: inf sign differs"
    fin = ~(nan_ref | inf_ref)
    zero = torch.zeros((), dtype=torch.float64, device=dev)
    err = torch.where(fin, (g - r).abs(), zero)
    mag = torch.where(fin, r.abs(), zero)
    if gpu.dtype == torch.bfloat16:
        tol, rel, quantum = BF16_TOL, BF16_TIGHT, 1.2e-38
    else:
        tol = DT_TOL[gpu.dtype]
        rel, quantum = DT_TIGHT[gpu.dtype]
    worst = float((err / (tol * mag.clamp(min=1.0))).max()) if err.numel() else 0.0
    assert worst <= 1.0, f"{what}: max err/bound = {worst:.3f}"
    if tight and err.numel():
        worst_t = float((err / (rel * mag + quantum)).max())
        assert worst_t <= 1.0, f"{what}: exceeds one-rounding bound by {worst_t:.3f}x"
    return worst


def assert_loss_close(gpu: torch.Tensor, ref: np.ndarray, what: str = ""):
    got = gpu.detach().cpu().double().numpy().reshape(ref.shape)
    nan_ref = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan_ref), f"{what}: NaN pattern differs"
    inf_ref = np.isinf(ref)
    assert np.array_equal(np.isinf(got), inf_ref), f"{what}: inf pattern differs"
    assert np.array_equal(got[inf_ref], ref[inf_ref]), f"{what}: inf sign differs"
    fin = ~(nan_ref | inf_ref)
    err = np.abs(got[fin] - ref[fin])
    bound = LOSS_TOL * np.maximum(1.0, np.abs(ref[fin]))
    worst = float(np.max(err / bound)) if err.size else 0.0
    assert worst <= 1.0, f"{what}: max loss err/bound = {worst:.3f}"
    return worst


def guarded(shape, dtype, device, pad_elems: int = 2048, fill: int = 0x5A):
    """Allocate ``shape`` inside a larger byte-filled buffer.  Returns (view, check) where
    check() asserts the pads before and after the view are untouched."""
    n = int(np.prod(shape))
    esz = torch.empty((), dtype=dtype).element_size()
    raw = torch.full(((n + 2 * pad_elems) * esz,), fill, dtype=torch.uint8, device=device)
    view = raw[pad_elems * esz:(pad_elems + n) * esz].view(dtype).view(shape)

    def check():
        head = raw[:pad_elems * esz]
        tail = raw[(pad_elems + n) * esz:]
        assert bool((head == fill).all()) and bool((tail == fill).all()), "write outside the output"

    return view, check

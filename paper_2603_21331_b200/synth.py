"""Seeded synthetic inputs for the three row-reduction ops.

This module holds NO arithmetic of the ops themselves; it only draws random tensors
with the shapes and value distributions of the benchmark workloads, so that the CUDA
library and the CPU checker can be fed the very same bf16 bit patterns.

Recipes (all values are drawn in float32 and rounded once to bf16, round-to-nearest-even):

* RMSNorm: x ~ N(0, 1); weight = 1 + 0.1 * N(0, 1).
* Softmax: x ~ N(0, 4^2) (attention-score-like); each row is causal-masked with
  probability 0.1: its last k entries become -inf, k uniform in {0, ..., D-1}.
* Cross-entropy: logits ~ N(0, 2^2); targets uniform in [0, V); each target is replaced
  by ``ignore_index`` with probability 0.05.
* Adversarial rows (Section 4, Stage 3 of the paper names "rows of large identical
  values" and "near-zero variance"): see :func:`adversarial_rows`.

A seed names a ``torch.Generator`` on the requested device.  CPU and CUDA generators
produce different streams; parity never depends on that because both sides always
receive the same generated bits.  Large tensors are drawn in row chunks so the float32
staging buffer stays small.
"""
from __future__ import annotations

import numpy as np
import torch

IGNORE_INDEX = -100
_CHUNK_ELEMS = 1 << 26  # float32 staging buffer of at most 256 MiB


def _gen(seed: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def _normal_bf16(rows: int, cols: int, std: float, mean: float, g: torch.Generator,
                 device, dtype=torch.bfloat16) -> torch.Tensor:
    out = torch.empty((rows, cols), dtype=dtype, device=device)
    step = max(1, _CHUNK_ELEMS // max(1, cols))
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        t = torch.randn((r1 - r0, cols), dtype=torch.float32, device=device, generator=g)
        if std != 1.0:
            t.mul_(std)
        if mean != 0.0:
            t.add_(mean)
        out[r0:r1].copy_(t)
    return out


def to_bits(t: torch.Tensor) -> np.ndarray:
    """bf16 tensor (any device) -> numpy uint16 array of its bit patterns."""
    if t.dtype != torch.bfloat16:
        raise TypeError("expected a bfloat16 tensor")
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def to_elems(t: torch.Tensor) -> np.ndarray:
    """Tensor of any supported element type -> the array the CPU checker's *_dt functions take:
    uint16 bit patterns for bf16 / fp16, float32 values for fp32."""
    t = t.detach().contiguous().cpu()
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).numpy().view(np.uint16)
    if t.dtype == torch.float32:
        return t.numpy()
    raise TypeError("expected a bfloat16, float16 or float32 tensor")


DTYPE_NAMES = {torch.bfloat16: "bf16", torch.float16: "f16", torch.float32: "f32"}


def from_bits(bits: np.ndarray, device="cpu") -> torch.Tensor:
    """numpy uint16 bit patterns -> bf16 tensor on ``device``."""
    a = np.ascontiguousarray(bits, dtype=np.uint16)
    return torch.from_numpy(a.view(np.int16).copy()).view(torch.bfloat16).to(device)


def rmsnorm_inputs(rows: int, D: int, seed: int, device="cpu", dtype=torch.bfloat16):
    """(x [rows, D], w [D]) of element type ``dtype`` (float32 draws rounded once to it)."""
    g = _gen(seed, device)
    x = _normal_bf16(rows, D, 1.0, 0.0, g, device, dtype)
    w = _normal_bf16(1, D, 0.1, 1.0, g, device, dtype).reshape(D)
    return x, w


def layernorm_inputs(rows: int, D: int, seed: int, device="cpu", dtype=torch.bfloat16):
    """(x bf16 [rows, D] ~ N(0.5, 1.5^2), gamma bf16 [D] = 1 + 0.1 N(0,1), beta bf16 [D] = 0.1 N(0,1)).
    The non-zero mean makes the centring matter."""
    g = _gen(seed, device)
    x = _normal_bf16(rows, D, 1.5, 0.5, g, device, dtype)
    gamma = _normal_bf16(1, D, 0.1, 1.0, g, device, dtype).reshape(D)
    beta = _normal_bf16(1, D, 0.1, 0.0, g, device, dtype).reshape(D)
    return x, gamma, beta


def rope_inputs(n_seq: int, S: int, Dh: int, seed: int, device="cpu", dtype=torch.bfloat16):
    """x [n_seq, S, Dh] ~ N(0, 1): query / key head vectors before the rotation."""
    g = _gen(seed, device)
    return _normal_bf16(n_seq * S, Dh, 1.0, 0.0, g, device, dtype).view(n_seq, S, Dh)


def softmax_inputs(rows: int, D: int, seed: int, device="cpu", mask_frac: float = 0.1,
                   dtype=torch.bfloat16):
    """x [rows, D] with ~mask_frac of the rows causal-masked by trailing -inf."""
    g = _gen(seed, device)
    x = _normal_bf16(rows, D, 4.0, 0.0, g, device, dtype)
    masked = torch.rand((rows,), device=device, generator=g) < mask_frac
    k = torch.randint(0, D, (rows,), device=device, generator=g)  # {0..D-1}
    k = torch.where(masked, k, torch.zeros_like(k))
    step = max(1, _CHUNK_ELEMS // max(1, D))
    cols = torch.arange(D, device=device)
    for r0 in range(0, rows, step):
        r1 = min(rows, r0 + step)
        m = cols[None, :] >= (D - k[r0:r1])[:, None]
        x[r0:r1].masked_fill_(m, float("-inf"))
    return x


def xent_inputs(rows: int, V: int, seed: int, device="cpu", ignore_frac: float = 0.05,
                ignore_index: int = IGNORE_INDEX, dtype=torch.bfloat16):
    """(logits [rows, V] of element type ``dtype``, targets int64 [rows])."""
    g = _gen(seed, device)
    logits = _normal_bf16(rows, V, 2.0, 0.0, g, device, dtype)
    targets = torch.randint(0, V, (rows,), dtype=torch.int64, device=device, generator=g)
    ign = torch.rand((rows,), device=device, generator=g) < ignore_frac
    targets = torch.where(ign, torch.full_like(targets, ignore_index), targets)
    return logits, targets


ADVERSARIAL_KINDS = ("big_equal", "alternating_big", "tiny", "mixed_extremes",
                     "all_equal", "one_huge")


def adversarial_rows(kind: str, rows: int, D: int, seed: int, device="cpu"):
    """Adversarial bf16 rows.  Returns (x bf16 [rows, D], hot int64 [rows]).

    ``hot[r]`` is the column of the planted extreme value for kind "one_huge" (else 0);
    cross-entropy tests aim the target at it for half of the rows.

    * big_equal        every entry +65000 (rounds to 65024 in bf16)
    * alternating_big  +65024, -65024, +65024, ...
    * tiny             entries +-1e-30 with random signs
    * mixed_extremes   N(0,1) with ~1% entries +-65024 and ~1% entries +-1e-30
    * all_equal        row r is constant c_r, c cycling through {0, 1, -3.5, 65024, 1e-30}
    * one_huge         N(0,1) with a single entry equal to 65024 per row
    """
    g = _gen(seed, device)
    hot = torch.zeros((rows,), dtype=torch.int64, device=device)
    if kind == "big_equal":
        x = torch.full((rows, D), 65000.0, dtype=torch.float32, device=device)
    elif kind == "alternating_big":
        sign = 1.0 - 2.0 * (torch.arange(D, device=device) % 2).to(torch.float32)
        x = (65024.0 * sign)[None, :].expand(rows, D).clone()
    elif kind == "tiny":
        sign = torch.where(torch.rand((rows, D), device=device, generator=g) < 0.5, -1.0, 1.0)
        x = 1e-30 * sign
    elif kind == "mixed_extremes":
        x = torch.randn((rows, D), dtype=torch.float32, device=device, generator=g)
        u = torch.rand((rows, D), device=device, generator=g)
        sign = torch.where(torch.rand((rows, D), device=device, generator=g) < 0.5, -1.0, 1.0)
        x = torch.where(u < 0.01, 65024.0 * sign, x)
        x = torch.where((u >= 0.01) & (u < 0.02), 1e-30 * sign, x)
    elif kind == "all_equal":
        consts = torch.tensor([0.0, 1.0, -3.5, 65024.0, 1e-30], dtype=torch.float32,
                              device=device)
        c = consts[torch.arange(rows, device=device) % consts.numel()]
        x = c[:, None].expand(rows, D).clone()
    elif kind == "one_huge":
        x = torch.randn((rows, D), dtype=torch.float32, device=device, generator=g)
        hot = torch.randint(0, D, (rows,), dtype=torch.int64, device=device, generator=g)
        x[torch.arange(rows, device=device), hot] = 65024.0
    else:
        raise ValueError(f"unknown adversarial kind {kind!r}")
    return x.to(torch.bfloat16), hot


def case_seed(config: int, case_index: int) -> int:
    """Seed convention: config 1 uses seed 0; otherwise 1000 * config + case index."""
    return 0 if config == 1 else 1000 * int(config) + int(case_index)

"""Pins for the checker's LayerNorm and row-sum (CPU only): closed forms, invariants, a
50-digit brute force of the definitions on tiny inputs and an fp64 library cross-check,
chosen so that a slip (unbiased variance, eps outside the root, beta scaled by gamma,
gamma indexed by row, missing centring) fails at least one of them."""
import math

import numpy as np
import pytest
import torch
from mpmath import mp, mpf

import oracle
from paper_2603_21331_b200 import synth
from test_oracle_pins import bits


def test_layernorm_1234_closed_form():
    # x = [1, 2, 3, 4]: mu = 2.5, biased var = 1.25; eps = 0 -> y = (x - 2.5) / sqrt(1.25)
    y = oracle.layernorm(bits([[1.0, 2.0, 3.0, 4.0]]), bits(np.ones(4)), bits(np.zeros(4)), 0.0)
    s = math.sqrt(1.25)
    assert np.allclose(y[0], [-1.5 / s, -0.5 / s, 0.5 / s, 1.5 / s], rtol=1e-15)
    # with eps: denominator sqrt(1.25 + eps32); gamma and beta per column
    eps32 = float(np.float32(1e-5))
    g = np.array([1.0, 0.5, 2.0, -1.0])
    b = np.array([0.25, -0.5, 0.0, 3.0])
    y = oracle.layernorm(bits([[1.0, 2.0, 3.0, 4.0]]), bits(g), bits(b), 1e-5)
    want = (np.array([1.0, 2.0, 3.0, 4.0]) - 2.5) / math.sqrt(1.25 + eps32) * g + b
    assert np.allclose(y[0], want, rtol=1e-14)
    # unbiased variance (divide by D-1) would give sqrt(5/3): make sure it is not that
    assert abs(y[0, 3] - (1.5 / math.sqrt(5.0 / 3.0 + eps32) * -1.0 + 3.0)) > 1e-2


@pytest.mark.parametrize("c", [0.0, 1.0, -3.5, 65024.0, 1e-30])
def test_layernorm_constant_row_gives_beta(c):
    D = 1537
    rng = np.random.default_rng(2)
    g = oracle.bf16_to_f64(bits(1.0 + 0.1 * rng.standard_normal(D)))
    b = oracle.bf16_to_f64(bits(0.1 * rng.standard_normal(D)))
    y = oracle.layernorm(bits(np.full((2, D), c)), bits(g), bits(b), 1e-5)
    assert np.array_equal(y, np.broadcast_to(b, (2, D)))


def test_layernorm_invariants():
    x, g, b = synth.layernorm_inputs(12, 4097, seed=61)
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    gd, bd = oracle.bf16_to_f64(gb), oracle.bf16_to_f64(bb)
    y0 = oracle.layernorm(xb, gb, bb, 0.0)
    z = (y0 - bd[None, :]) / gd[None, :]
    assert np.allclose(z.mean(axis=1), 0.0, atol=1e-13)            # centred
    assert np.allclose((z * z).mean(axis=1), 1.0, rtol=1e-12)       # unit variance at eps = 0
    # shift by an exactly representable amount and scale by a power of two leave y unchanged
    xq = torch.round(x.float() * 4) / 4                             # multiples of 1/4
    xq = xq.clamp(-8, 8).to(torch.bfloat16)
    ya = oracle.layernorm(synth.to_bits(xq), gb, bb, 0.0)
    yb_ = oracle.layernorm(synth.to_bits((xq.float() + 16.0).to(torch.bfloat16)), gb, bb, 0.0)
    assert np.array_equal(oracle.bf16_to_f64(synth.to_bits((xq.float() + 16.0).to(torch.bfloat16))),
                          oracle.bf16_to_f64(synth.to_bits(xq)) + 16.0)
    assert np.max(np.abs(ya - yb_)) < 1e-12
    yc = oracle.layernorm(synth.to_bits((xq.float() * 4.0).to(torch.bfloat16)), gb, bb, 0.0)
    assert np.max(np.abs(ya - yc)) < 1e-12
    # eps matters: with eps > 0 the normalised values shrink by sqrt(var / (var + eps))
    y1 = oracle.layernorm(xb, gb, bb, 1.0)
    xd = oracle.bf16_to_f64(xb)
    var = xd.var(axis=1)
    z1 = (y1 - bd[None, :]) / gd[None, :]
    assert np.allclose((z1 * z1).mean(axis=1), var / (var + 1.0), rtol=1e-12)


def test_layernorm_brute_force_4x8():
    mp.dps = 50
    rng = np.random.default_rng(7)
    x = rng.integers(-20, 21, size=(4, 8)) * 0.25
    g = rng.integers(2, 9, size=8) * 0.25
    b = rng.integers(-4, 5, size=8) * 0.5
    eps32 = float(np.float32(1e-5))
    y = oracle.layernorm(bits(x), bits(g), bits(b), 1e-5)
    for r in range(4):
        xs = [mpf(float(v)) for v in x[r]]
        mu = sum(xs) / 8
        var = sum((v - mu) ** 2 for v in xs) / 8
        den = mp.sqrt(var + mpf(eps32))
        for j in range(8):
            want = (xs[j] - mu) / den * mpf(float(g[j])) + mpf(float(b[j]))
            assert abs(mpf(float(y[r, j])) - want) < mpf("1e-13")


@pytest.mark.parametrize("rows,D", [(5, 1), (7, 8), (33, 1023), (9, 4097)])
def test_layernorm_and_rowsum_against_torch_fp64(rows, D):
    import torch.nn.functional as F
    x, g, b = synth.layernorm_inputs(rows, D, seed=71)
    got = oracle.layernorm(synth.to_bits(x), synth.to_bits(g), synth.to_bits(b), 1e-5)
    want = F.layer_norm(x.double(), (D,), g.double(), b.double(), float(np.float32(1e-5))).numpy()
    assert np.allclose(got, want, rtol=1e-11, atol=1e-12)
    s = oracle.rowsum(synth.to_bits(x))
    assert np.allclose(s, x.double().sum(dim=-1).numpy(), rtol=1e-13, atol=1e-12)


def test_rowsum_closed_forms_and_exactness():
    # 1 + 2 + ... + 100 = 5050; alternating +-65024 cancels exactly; constants give c * D
    x = np.arange(1, 101, dtype=np.float64)[None, :]
    assert oracle.rowsum(bits(x))[0] == 5050.0
    alt = np.where(np.arange(4096) % 2 == 0, 65024.0, -65024.0)[None, :]
    assert oracle.rowsum(bits(alt))[0] == 0.0
    for c, D in ((0.25, 4099), (-3.5, 7), (65024.0, 16384)):
        assert oracle.rowsum(bits(np.full((3, D), c)))[1] == c * D
    # integers in bf16 sum exactly in double: compare with Python's exact integer sum
    rng = np.random.default_rng(11)
    v = rng.integers(-128, 129, size=(6, 4097))
    assert np.array_equal(oracle.rowsum(bits(v.astype(np.float64))), v.sum(axis=1).astype(np.float64))
    # linearity in the rows: sum of two rows' sums equals the sum of the concatenation
    a = oracle.rowsum(bits(v[:1].astype(np.float64)))[0] + oracle.rowsum(bits(v[1:2].astype(np.float64)))[0]
    assert a == oracle.rowsum(bits(np.concatenate([v[0], v[1]])[None, :].astype(np.float64)))[0]

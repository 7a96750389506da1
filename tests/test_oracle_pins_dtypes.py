"""Pins for the checker's element-type variants (CPU only).  The bf16 functions are pinned
elsewhere; here the fp16 / fp32 loaders are pinned against known bit patterns and numpy's own
half type, the *_dt functions are tied to the pinned bf16 ones on inputs every type holds
exactly, and closed forms and an fp64 library cross-check cover values only fp16 / fp32 hold."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from paper_2603_21331_b200 import synth
from test_oracle_pins import bits


def test_f16_widening_known_patterns_and_all_65536_against_numpy():
    known = {0x0000: 0.0, 0x3C00: 1.0, 0xC000: -2.0, 0x7BFF: 65504.0, 0x0001: 2.0 ** -24,
             0x03FF: 1023 * 2.0 ** -24, 0x0400: 2.0 ** -14, 0x3555: 0.333251953125,
             0x7C00: math.inf, 0xFC00: -math.inf}
    got = oracle.f16_to_f64(np.array(list(known), dtype=np.uint16))
    assert np.array_equal(got, np.array(list(known.values())))
    assert math.copysign(1.0, oracle.f16_to_f64(np.array([0x8000], dtype=np.uint16))[0]) == -1.0
    allb = np.arange(65536, dtype=np.uint16)
    got = oracle.f16_to_f64(allb)
    want = allb.view(np.float16).astype(np.float64)
    nan = np.isnan(want)
    assert np.array_equal(np.isnan(got), nan) and nan.sum() == 2 * 1023
    assert np.array_equal(got[~nan], want[~nan]) and np.array_equal(np.signbit(got[~nan]), np.signbit(want[~nan]))


def _as(dtype, a):
    t = torch.from_numpy(np.asarray(a, dtype=np.float64)).to({"bf16": torch.bfloat16, "f16": torch.float16,
                                                             "f32": torch.float32}[dtype])
    assert np.array_equal(t.double().numpy(), np.asarray(a, dtype=np.float64)), "value not representable"
    return synth.to_elems(t)


def test_dt_functions_agree_with_the_pinned_bf16_functions_on_shared_values():
    # multiples of 1/8 in [-16, 16] are exact in bf16, fp16 and fp32: all element types must
    # then give the very same doubles, and those of the bf16 entry points
    rng = np.random.default_rng(5)
    x = rng.integers(-128, 129, size=(6, 37)) / 8.0
    w = rng.integers(4, 13, size=37) / 8.0
    t = rng.integers(0, 37, size=6).astype(np.int64)
    t[2] = -100
    base_r = oracle.rmsnorm(bits(x), bits(w), 1e-6)
    base_s = oracle.softmax(bits(x))
    base_x = oracle.xent(bits(x), t)
    for dt in ("bf16", "f16", "f32"):
        assert np.array_equal(oracle.rmsnorm_dt(_as(dt, x), _as(dt, w), 1e-6, dt), base_r)
        assert np.array_equal(oracle.softmax_dt(_as(dt, x), dt), base_s)
        lr, lm, n = oracle.xent_dt(_as(dt, x), t, dt)
        assert np.array_equal(lr, base_x[0]) and lm == base_x[1] and n == base_x[2] == 5


def test_layernorm_and_rowsum_dt_agree_with_the_pinned_bf16_functions_and_torch():
    rng = np.random.default_rng(6)
    x = rng.integers(-128, 129, size=(5, 41)) / 8.0
    g = rng.integers(4, 13, size=41) / 8.0
    b = rng.integers(-8, 9, size=41) / 8.0
    base_l = oracle.layernorm(bits(x), bits(g), bits(b), 1e-5)
    base_s = oracle.rowsum(bits(x))
    for dt in ("bf16", "f16", "f32"):
        assert np.array_equal(oracle.layernorm_dt(_as(dt, x), _as(dt, g), _as(dt, b), 1e-5, dt), base_l)
        assert np.array_equal(oracle.rowsum_dt(_as(dt, x), dt), base_s)
    # values only fp16 / fp32 hold: a row of c and c + 2^-10 alternating has mean c + 2^-11,
    # deviations +-2^-11, variance 2^-22: y = +-1 / sqrt(1 + eps / 2^-22) exactly in closed form
    eps32 = float(np.float32(1e-5))
    for dt in ("f16", "f32"):
        row = np.where(np.arange(64) % 2 == 0, 1.0, 1.0 + 2.0 ** -10)[None, :]
        y = oracle.layernorm_dt(_as(dt, row), _as(dt, np.ones(64)), _as(dt, np.zeros(64)), 1e-5, dt)
        want = np.where(np.arange(64) % 2 == 0, -1.0, 1.0) * 2.0 ** -11 / math.sqrt(2.0 ** -22 + eps32)
        assert np.allclose(y[0], want, rtol=1e-12)
        assert oracle.rowsum_dt(_as(dt, row), dt)[0] == 64 + 32 * 2.0 ** -10
    for dt, tdt in (("f16", torch.float16), ("f32", torch.float32)):
        x, g, b = synth.layernorm_inputs(9, 1537, seed=84, dtype=tdt)
        got = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, dt)
        want = F.layer_norm(x.double(), (1537,), g.double(), b.double(), float(np.float32(1e-5))).numpy()
        assert np.allclose(got, want, rtol=1e-11, atol=1e-12)
        assert np.allclose(oracle.rowsum_dt(synth.to_elems(x), dt), x.double().sum(dim=-1).numpy(), rtol=1e-13)


def test_dt_closed_forms_on_values_only_wider_types_hold():
    # c = 1 + 2^-10 (fp16, fp32) and 1 + 2^-20 (fp32 only): constant rows
    eps32 = float(np.float32(1e-6))
    for dt, c in (("f16", 1.0 + 2.0 ** -10), ("f32", 1.0 + 2.0 ** -10), ("f32", 1.0 + 2.0 ** -20)):
        x = np.full((2, 9), c)
        w = np.full(9, 0.5)
        y = oracle.rmsnorm_dt(_as(dt, x), _as(dt, w), 1e-6, dt)
        assert np.allclose(y, c * 0.5 / math.sqrt(c * c + eps32), rtol=1e-15)
        # all-equal rows: softmax 1/D, loss log D
        assert np.allclose(oracle.softmax_dt(_as(dt, x), dt), 1.0 / 9.0, rtol=1e-15)
        lr, lm, n = oracle.xent_dt(_as(dt, x), np.array([0, 8], dtype=np.int64), dt)
        assert np.allclose(lr, math.log(9.0), rtol=1e-15) and n == 2
    # two-element softmax = sigmoid of the difference; the difference 2^-11 needs fp16's / fp32's bits
    for dt in ("f16", "f32"):
        a = 1.0 + 2.0 ** -10
        y = oracle.softmax_dt(_as(dt, [[1.0, a]]), dt)
        assert abs(y[0, 1] - 1.0 / (1.0 + math.exp(-(2.0 ** -10)))) < 1e-16
        lr, _, _ = oracle.xent_dt(_as(dt, [[1.0, a]]), np.array([0], dtype=np.int64), dt)
        assert abs(lr[0] - math.log1p(math.exp(2.0 ** -10))) < 1e-15
    # fp16 range: 65504 and the smallest subnormal in one row
    y = oracle.rmsnorm_dt(_as("f16", [[65504.0, 2.0 ** -24]]), _as("f16", [1.0, 1.0]), 0.0, "f16")
    rms = math.sqrt((65504.0 ** 2 + 2.0 ** -48) / 2.0)
    assert np.allclose(y[0], [65504.0 / rms, 2.0 ** -24 / rms], rtol=1e-15)


@pytest.mark.parametrize("dt,tdt", [("f16", torch.float16), ("f32", torch.float32)])
@pytest.mark.parametrize("rows,D", [(5, 1), (7, 8), (33, 1023), (9, 4097)])
def test_dt_functions_against_torch_fp64(dt, tdt, rows, D):
    x, w = synth.rmsnorm_inputs(rows, D, seed=81, dtype=tdt)
    got = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 1e-6, dt)
    xd = x.double()
    want = (xd / torch.sqrt((xd * xd).mean(dim=-1, keepdim=True) + float(np.float32(1e-6))) * w.double()).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=0)
    xs = synth.softmax_inputs(rows, D, seed=82, mask_frac=0.3, dtype=tdt)
    got = oracle.softmax_dt(synth.to_elems(xs), dt)
    assert np.allclose(got, F.softmax(xs.double(), dim=-1).numpy(), rtol=1e-12, atol=1e-300)
    lg, tg = synth.xent_inputs(rows, D, seed=83, dtype=tdt)
    lr, lm, n = oracle.xent_dt(synth.to_elems(lg), tg.numpy(), dt)
    want = F.cross_entropy(lg.double(), tg, ignore_index=-100, reduction="none").numpy()
    assert np.allclose(lr, want, rtol=1e-12, atol=1e-13)
    if n > 0:
        assert abs(lm - F.cross_entropy(lg.double(), tg, ignore_index=-100).item()) < 1e-12

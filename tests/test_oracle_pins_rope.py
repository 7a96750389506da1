"""Pins for the checker's rotary embedding (CPU only): 40-digit closed forms, invariants, a
50-digit brute force and an fp64 library cross-check through complex multiplication, chosen so
that a slip (exponent i/Dh instead of 2i/Dh, rotate-half pairing, wrong sign of the sine,
position taken from the wrong axis, offset ignored) fails at least one of them."""
import numpy as np
import pytest
import torch
from mpmath import mp, mpf

import oracle
from paper_2603_21331_b200 import synth
from test_oracle_pins import GOLD


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def test_rope_closed_forms_pair0_and_the_square_root_pair():
    # Dh = 4, base = 1e4: pair 0 turns by p, pair 1 by p / 100; x = (1, 0, 0, 1) at positions 0..2047
    S = 2048
    x = _f32(np.tile([1.0, 0.0, 0.0, 1.0], (1, S, 1)))
    y = oracle.rope(x, "f32")
    assert np.array_equal(y[0, 0], [1.0, 0.0, 0.0, 1.0])                      # position 0: identity
    for p in (1, 2, 3, 2047):
        assert abs(y[0, p, 0] - GOLD[f"cos_{p}"]) < 1e-15 and abs(y[0, p, 1] - GOLD[f"sin_{p}"]) < 1e-15
        # the second pair starts on the y axis: (0, 1) -> (-sin, cos)
        assert abs(y[0, p, 2] + GOLD[f"sin_{p}_over_100"]) < 1e-14   # angle p * 1e4^-0.5 carries a double rounding
        assert abs(y[0, p, 3] - GOLD[f"cos_{p}_over_100"]) < 1e-14
    # Dh = 128: pair 16 has exponent -32/128 = -1/4, i.e. angle p / 10
    x = np.zeros((1, 8, 128), dtype=np.float32)
    x[0, :, 32] = 1.0
    y = oracle.rope(x, "f32")
    assert abs(y[0, 7, 32] - GOLD["cos_7_over_10"]) < 1e-15 and abs(y[0, 7, 33] - GOLD["sin_7_over_10"]) < 1e-15
    assert np.count_nonzero(y[0, 7]) == 2                                     # nothing leaks into other pairs


def test_rope_offset_sequence_axis_and_base():
    x = synth.rope_inputs(3, 5, 8, seed=31, dtype=torch.float32)
    xe = synth.to_elems(x)
    y = oracle.rope(xe, "f32", pos_offset=0)
    # positions run along axis 1 and restart for every sequence of axis 0
    for n in range(3):
        assert np.array_equal(oracle.rope(xe[n:n + 1], "f32"), y[n:n + 1])
    # an offset shifts the positions: the vectors of rows 2..4 alone, started at offset 2
    assert np.array_equal(oracle.rope(xe[:, 2:5], "f32", pos_offset=2), y[:, 2:5])
    assert not np.allclose(oracle.rope(xe[:, 2:5], "f32", pos_offset=0), y[:, 2:5])
    # base = 1 makes every pair turn by p itself
    y1 = oracle.rope(xe, "f32", base=1.0)
    p = np.arange(5)[None, :, None]
    a, b = xe[:, :, 0::2].astype(np.float64), xe[:, :, 1::2].astype(np.float64)
    assert np.allclose(y1[:, :, 0::2], a * np.cos(p) - b * np.sin(p), rtol=0, atol=1e-15)
    assert np.allclose(y1[:, :, 1::2], a * np.sin(p) + b * np.cos(p), rtol=0, atol=1e-15)


def test_rope_invariants():
    x = synth.rope_inputs(2, 33, 64, seed=32, dtype=torch.float32)
    xe = synth.to_elems(x)
    xd = xe.astype(np.float64)
    y = oracle.rope(xe, "f32")
    # a rotation keeps the length of every pair, hence of every head vector
    n_in = xd[:, :, 0::2] ** 2 + xd[:, :, 1::2] ** 2
    n_out = y[:, :, 0::2] ** 2 + y[:, :, 1::2] ** 2
    assert np.allclose(n_in, n_out, rtol=1e-14)
    # and the relative-position property: <rope(q, m), rope(k, n)> depends on m - n only
    q, k = xe[0:1], xe[1:2]
    d1 = (oracle.rope(q, "f32", pos_offset=5) * oracle.rope(k, "f32", pos_offset=2)).sum(axis=-1)
    d2 = (oracle.rope(q, "f32", pos_offset=103) * oracle.rope(k, "f32", pos_offset=100)).sum(axis=-1)
    assert np.allclose(d1, d2, rtol=0, atol=1e-11)
    # linearity: rope(2x) = 2 rope(x)
    assert np.array_equal(oracle.rope(_f32(2 * xe), "f32"), 2 * y)


def test_rope_brute_force_50_digits():
    mp.dps = 50
    rng = np.random.default_rng(9)
    x = _f32(rng.integers(-16, 17, size=(2, 3, 6)) / 4.0)
    y = oracle.rope(x, "f32", base=10000.0, pos_offset=11)
    for n in range(2):
        for s in range(3):
            for i in range(3):
                th = mpf(11 + s) * mp.power(mpf(10000), -mpf(2 * i) / 6)
                a, b = mpf(float(x[n, s, 2 * i])), mpf(float(x[n, s, 2 * i + 1]))
                assert abs(mpf(float(y[n, s, 2 * i])) - (a * mp.cos(th) - b * mp.sin(th))) < mpf("1e-14")
                assert abs(mpf(float(y[n, s, 2 * i + 1])) - (a * mp.sin(th) + b * mp.cos(th))) < mpf("1e-14")


@pytest.mark.parametrize("dt,tdt", [("bf16", torch.bfloat16), ("f16", torch.float16), ("f32", torch.float32)])
@pytest.mark.parametrize("n_seq,S,Dh", [(1, 1, 2), (3, 17, 8), (2, 129, 128), (4, 33, 96)])
def test_rope_against_torch_complex_fp64(dt, tdt, n_seq, S, Dh):
    x = synth.rope_inputs(n_seq, S, Dh, seed=33, dtype=tdt)
    got = oracle.rope(synth.to_elems(x), dt, pos_offset=3)
    inv = 10000.0 ** (-torch.arange(0, Dh, 2, dtype=torch.float64) / Dh)
    ang = torch.outer(torch.arange(3, 3 + S, dtype=torch.float64), inv)
    z = torch.view_as_complex(x.double().reshape(n_seq, S, Dh // 2, 2).contiguous()) * torch.polar(
        torch.ones_like(ang), ang)
    want = torch.view_as_real(z).reshape(n_seq, S, Dh).numpy()
    assert np.allclose(got, want, rtol=0, atol=1e-12)

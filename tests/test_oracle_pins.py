"""Pins the fp64 CPU checker to things it did not compute itself (CPU only).

Closed forms (tests/golden/closed_forms.txt, 40-digit mpmath), invariants, special cases
that reduce to textbook formulas, a 50-digit brute force of the *naive* definitions on
tiny inputs, and an fp64 library cross-check.  Each family is chosen so that a plausible
slip in the checker (dropped term, wrong divisor, eps outside the root, weight indexed
by row, wrong sign, base-2 log, off-by-one target) fails at least one test.
"""
import math
import os
import struct

import numpy as np
import pytest
import torch
from mpmath import mp, mpf

import oracle
from paper_2603_21331_b200 import synth

GOLD = {}
with open(os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")) as _f:
    for _line in _f:
        if _line.startswith("#") or not _line.strip():
            continue
        _name, _val = _line.split("#")[0].split()
        GOLD[_name] = float(_val)


def bits(values) -> np.ndarray:
    """float values -> bf16 bit patterns (round-to-nearest-even), independent helper
    written with struct arithmetic rather than torch."""
    flat = np.asarray(values, dtype=np.float64).ravel()
    out = np.empty(flat.shape, dtype=np.uint16)
    for i, v in enumerate(flat):
        u = struct.unpack("<I", struct.pack("<f", float(v)))[0]
        if (u & 0x7F800000) == 0x7F800000:        # inf / nan: truncate
            out[i] = u >> 16
            continue
        lsb = (u >> 16) & 1
        u = (u + 0x7FFF + lsb) & 0xFFFFFFFF
        out[i] = u >> 16
    return out.reshape(np.asarray(values).shape)


# --------------------------------------------------------------------------- bf16 widening
def test_bf16_widening_known_patterns():
    pats = np.array([0x3F80, 0xBF80, 0x0000, 0x8000, 0xC2C8, 0x477E, 0xFF80, 0x7F80, 0x3E80],
                    dtype=np.uint16)
    got = oracle.bf16_to_f64(pats)
    want = [1.0, -1.0, 0.0, -0.0, -100.0, 65024.0, -math.inf, math.inf, 0.25]
    assert got.tolist() == want
    assert math.copysign(1.0, got[3]) == -1.0
    assert math.isnan(oracle.bf16_to_f64(np.array([0x7FC0], dtype=np.uint16))[0])
    # 65000 and 1e-30 land on the bf16 values the closed-form file states
    assert oracle.bf16_to_f64(bits([65000.0]))[0] == GOLD["bf16_of_65000"]
    assert oracle.bf16_to_f64(bits([1e-30]))[0] == pytest.approx(GOLD["bf16_of_1e-30"], rel=1e-15)
    # the struct-based rounding helper agrees with torch's RNE conversion
    v = torch.randn(4096, generator=torch.Generator().manual_seed(1)) * 37.0
    assert np.array_equal(bits(v.numpy()), synth.to_bits(v.to(torch.bfloat16)))


# --------------------------------------------------------------------------- softmax
def test_softmax_two_logits_is_sigmoid():
    y = oracle.softmax(bits([[1.0, 0.0]]))
    assert y[0, 0] == pytest.approx(GOLD["softmax2_1_0_first"], abs=1e-15)
    assert y[0, 1] == pytest.approx(GOLD["softmax2_1_0_second"], abs=1e-15)
    # orientation: a larger logit gets the larger probability
    y = oracle.softmax(bits([[0.0, 1.0]]))
    assert y[0, 1] > y[0, 0]


def test_softmax_invariants_random():
    x = synth.softmax_inputs(64, 1537, seed=11)
    xb = synth.to_bits(x)
    y = oracle.softmax(xb)
    assert np.all(np.abs(y.sum(axis=1) - 1.0) <= 1e-12)
    assert np.all((y >= 0.0) & (y <= 1.0))
    neg_inf = xb == 0xFF80
    assert neg_inf.any()
    assert np.all(y[neg_inf] == 0.0)
    # argmax is preserved, ordering is monotone
    xd = oracle.bf16_to_f64(xb)
    assert np.array_equal(y.argmax(axis=1), xd.argmax(axis=1))
    # ratio of two outputs equals exp of the logit difference
    r = 5
    i, j = 3, 17
    assert y[r, i] / y[r, j] == pytest.approx(math.exp(xd[r, i] - xd[r, j]), rel=1e-12)


def test_softmax_shift_invariance():
    # multiples of 1/4 in [-8, 8] shifted by 32 stay exactly representable in bf16
    rng = np.random.default_rng(5)
    base = rng.integers(-32, 33, size=(8, 33)) / 4.0
    y0 = oracle.softmax(bits(base))
    y1 = oracle.softmax(bits(base + 32.0))
    assert np.array_equal(oracle.bf16_to_f64(bits(base + 32.0)), base + 32.0)
    assert np.max(np.abs(y0 - y1)) <= 1e-15


@pytest.mark.parametrize("D", [1, 7, 4099])
@pytest.mark.parametrize("c", [0.0, 1.0, -3.5, 65024.0, 1e-30])
def test_softmax_all_equal_row(D, c):
    y = oracle.softmax(bits(np.full((2, D), c)))
    assert np.allclose(y, 1.0 / D, rtol=1e-13, atol=0)


def test_softmax_unpinned_conventions():
    # documented PyTorch conventions (not pinned by the paper): all -inf row -> NaN
    y = oracle.softmax(np.full((1, 5), 0xFF80, dtype=np.uint16))
    assert np.all(np.isnan(y))
    y = oracle.softmax(np.array([[0x7FC0, 0x3F80, 0x0000]], dtype=np.uint16))
    assert np.all(np.isnan(y))


# --------------------------------------------------------------------------- rmsnorm
def test_rmsnorm_3_4():
    y = oracle.rmsnorm(bits([[3.0, 4.0]]), bits([1.0, 1.0]), 0.0)
    assert y[0, 0] == pytest.approx(GOLD["rmsnorm_3_4_first"], rel=1e-15)
    assert y[0, 1] == pytest.approx(GOLD["rmsnorm_3_4_second"], rel=1e-15)


def test_rmsnorm_constant_rows_closed_form():
    D = 1023
    y = oracle.rmsnorm(bits(np.full((1, D), 2.0)), bits(np.full(D, 1.5)), 1e-6)
    assert np.allclose(y, GOLD["rmsnorm_const_2_w1p5"], rtol=1e-14, atol=0)
    y = oracle.rmsnorm(bits(np.full((1, D), -2.0)), bits(np.full(D, 1.5)), 1e-6)
    assert np.allclose(y, -GOLD["rmsnorm_const_2_w1p5"], rtol=1e-14, atol=0)
    # near-zero variance: eps dominates (eps inside the root, divisor D not D-1)
    y = oracle.rmsnorm(bits(np.full((1, D), 1e-30)), bits(np.ones(D)), 1e-6)
    assert np.allclose(y, GOLD["rmsnorm_const_tiny"], rtol=1e-13, atol=0)
    # general closed form w * sign(c) * |c| / sqrt(c^2 + eps), per-column weights
    rng = np.random.default_rng(3)
    w = oracle.bf16_to_f64(bits(1.0 + 0.1 * rng.standard_normal(D)))
    eps = float(np.float32(1e-6))
    for c in (0.0, 1.0, -3.5, 65024.0):
        y = oracle.rmsnorm(bits(np.full((3, D), c)), bits(w), 1e-6)
        want = w * c / math.sqrt(c * c + eps)
        assert np.allclose(y, want[None, :], rtol=1e-13, atol=0)


def test_rmsnorm_scale_invariance_and_unit_rms():
    x, w = synth.rmsnorm_inputs(16, 4097, seed=21)
    xb, wb = synth.to_bits(x), synth.to_bits(w)
    y = oracle.rmsnorm(xb, wb, 0.0)
    wd = oracle.bf16_to_f64(wb)
    # sum_j (y_j / w_j)^2 == D at eps = 0
    assert np.allclose(((y / wd[None, :]) ** 2).sum(axis=1), 4097.0, rtol=1e-12)
    # scaling the input by a power of two (exact in bf16) leaves y unchanged; by -1 flips it
    x4 = synth.to_bits(x * 4.0)
    assert np.max(np.abs(oracle.rmsnorm(x4, wb, 0.0) - y)) <= 1e-13
    xm = synth.to_bits(-x)
    assert np.max(np.abs(oracle.rmsnorm(xm, wb, 0.0) + y)) <= 1e-13
    # eps matters when it should: with eps > 0 the output shrinks
    y_eps = oracle.rmsnorm(xb, wb, 1.0)
    assert np.all(np.abs(y_eps) <= np.abs(y) + 1e-15) and np.any(np.abs(y_eps) < np.abs(y))
    # eps is taken as float32: 1e-6 as double would differ in the 9th digit
    one = oracle.rmsnorm(bits(np.full((1, 4), 1e-3)), bits(np.ones(4)), 1e-6)
    eps32 = float(np.float32(1e-6))
    c = oracle.bf16_to_f64(bits([1e-3]))[0]
    assert one[0, 0] == pytest.approx(c / math.sqrt(c * c + eps32), rel=1e-14)
    assert one[0, 0] != pytest.approx(c / math.sqrt(c * c + 1e-6), rel=1e-12)


# --------------------------------------------------------------------------- cross-entropy
def test_xent_two_logits_softplus():
    loss, mean, n = oracle.xent(bits([[1.0, 0.0], [1.0, 0.0]]), np.array([0, 1]))
    assert loss[0] == pytest.approx(GOLD["xent2_1_0_t0"], rel=1e-15)
    assert loss[1] == pytest.approx(GOLD["xent2_1_0_t1"], rel=1e-15)
    assert n == 2
    assert mean == pytest.approx((GOLD["xent2_1_0_t0"] + GOLD["xent2_1_0_t1"]) / 2, rel=1e-15)


@pytest.mark.parametrize("V", [8, 32000, 50304, 128256, 128257])
@pytest.mark.parametrize("c", [0.0, -3.5, 65024.0])
def test_xent_all_equal_is_log_V(V, c):
    x = bits(np.full((2, V), c))
    loss, mean, n = oracle.xent(x, np.array([0, V - 1]))
    assert np.allclose(loss, GOLD[f"log_{V}"], rtol=1e-13, atol=0)
    assert mean == pytest.approx(GOLD[f"log_{V}"], rel=1e-13)


def test_xent_dominant_logit():
    row = np.zeros(8)
    row[5] = 20.0
    loss, _, _ = oracle.xent(bits([row, row]), np.array([5, 2]))
    assert loss[0] == pytest.approx(GOLD["xent_hot_gap20_V8"], rel=1e-12)
    assert loss[1] == pytest.approx(GOLD["xent_cold_gap20_V8"], rel=1e-15)
    # gap of 65024: exactly 0 on the hot index, the gap elsewhere
    x, hot = synth.adversarial_rows("one_huge", 6, 257, seed=9)
    xb = synth.to_bits(x)
    xd = oracle.bf16_to_f64(xb)
    cold = (hot.numpy() + 1) % 257
    loss_hot, _, _ = oracle.xent(xb, hot.numpy())
    loss_cold, _, _ = oracle.xent(xb, cold)
    assert np.all(loss_hot == 0.0)
    assert np.allclose(loss_cold, 65024.0 - xd[np.arange(6), cold], rtol=1e-15)


def test_xent_matches_minus_log_softmax_and_is_nonnegative():
    logits, targets = synth.xent_inputs(48, 4099, seed=31, ignore_frac=0.0)
    xb, t = synth.to_bits(logits), targets.numpy()
    loss, mean, n = oracle.xent(xb, t)
    p = oracle.softmax(xb)
    assert np.allclose(loss, -np.log(p[np.arange(48), t]), rtol=1e-12, atol=1e-14)
    assert np.all(loss >= 0.0)
    assert n == 48 and mean == pytest.approx(loss.mean(), rel=1e-14)
    # expected magnitude for N(0, 2^2) logits: about log V + sigma^2/2 - E[x_t] = log V + 2
    assert abs(mean - (math.log(4099) + 2.0)) < 0.6


def test_xent_ignore_index_rows_contribute_nothing():
    logits, targets = synth.xent_inputs(200, 513, seed=32, ignore_frac=0.3)
    xb, t = synth.to_bits(logits), targets.numpy()
    keep = t != synth.IGNORE_INDEX
    assert 0 < keep.sum() < 200
    loss, mean, n = oracle.xent(xb, t)
    assert n == int(keep.sum())
    assert np.all(loss[~keep] == 0.0)
    loss2, mean2, n2 = oracle.xent(xb[keep], t[keep])
    assert n2 == n and mean2 == pytest.approx(mean, rel=1e-14)
    assert np.array_equal(loss2, loss[keep])
    assert mean * n == pytest.approx(loss.sum(), rel=1e-13)
    # a NaN planted in an ignored row must not leak
    xb2 = xb.copy()
    xb2[np.flatnonzero(~keep)[0], 7] = 0x7FC0
    loss3, mean3, _ = oracle.xent(xb2, t)
    assert mean3 == mean and np.array_equal(loss3, loss)
    # a different ignore_index value is honoured, and -100 then counts as out of range
    loss4, mean4, n4 = oracle.xent(xb, np.where(keep, t, 7), ignore_index=7)
    assert n4 == int((np.where(keep, t, 7) != 7).sum())


def test_xent_unpinned_conventions():
    xb = bits(np.zeros((3, 4)))
    loss, mean, n = oracle.xent(xb, np.array([-100, -100, -100]))
    assert n == 0 and math.isnan(mean) and np.all(loss == 0.0)
    loss, mean, n = oracle.xent(xb, np.array([0, 4, -1]))
    assert n == 3 and math.isnan(mean)
    assert loss[0] == pytest.approx(math.log(4)) and math.isnan(loss[1]) and math.isnan(loss[2])
    loss, mean, n = oracle.xent(bits(np.zeros((0, 4))), np.zeros((0,), dtype=np.int64))
    assert n == 0 and math.isnan(mean)


# --------------------------------------------------------------------------- brute force
def test_brute_force_4x8_naive_definitions():
    """Naive formulas (no max subtraction) in 50-digit arithmetic, straight-line code."""
    mp.dps = 50
    rng = np.random.default_rng(42)
    x = rng.integers(-20, 21, size=(4, 8)) * 0.25       # bf16-exact
    w = rng.integers(2, 9, size=8) * 0.25               # distinct per column
    t = np.array([0, 7, 3, 5])
    xb, wb = bits(x), bits(w)
    eps32 = float(np.float32(1e-6))
    sm = oracle.softmax(xb)
    rn = oracle.rmsnorm(xb, wb, 1e-6)
    loss, mean, n = oracle.xent(xb, t)
    total = mpf(0)
    for r in range(4):
        e = [mp.exp(mpf(float(v))) for v in x[r]]
        z = sum(e)
        ss = sum(mpf(float(v)) ** 2 for v in x[r])
        denom = mp.sqrt(ss / 8 + mpf(eps32))
        for j in range(8):
            assert abs(mpf(float(sm[r, j])) - e[j] / z) < mpf("1e-13")
            assert abs(mpf(float(rn[r, j])) - mpf(float(x[r, j])) * mpf(float(w[j])) / denom) < mpf("1e-13")
        lr = mp.log(z) - mpf(float(x[r, t[r]]))
        assert abs(mpf(float(loss[r])) - lr) < mpf("1e-13")
        total += lr
    assert abs(mpf(mean) - total / 4) < mpf("1e-13") and n == 4


# --------------------------------------------------------------------------- library cross-check
@pytest.mark.parametrize("rows,D", [(5, 1), (7, 8), (33, 1023), (9, 4097)])
def test_against_torch_fp64(rows, D):
    import torch.nn.functional as F
    x, w = synth.rmsnorm_inputs(rows, D, seed=77)
    xd, wd = x.double(), w.double()
    eps32 = float(np.float32(1e-6))
    got = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
    want = F.rms_norm(xd, (D,), wd, eps32).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=1e-300)

    xs = synth.softmax_inputs(rows, D, seed=78, mask_frac=0.5)
    got = oracle.softmax(synth.to_bits(xs))
    want = F.softmax(xs.double(), dim=-1).numpy()
    assert np.allclose(got, want, rtol=1e-12, atol=1e-300)

    logits, targets = synth.xent_inputs(rows, D, seed=79, ignore_frac=0.3)
    if (targets != -100).sum() == 0:
        targets[0] = 0
    loss, mean, n = oracle.xent(synth.to_bits(logits), targets.numpy())
    want_rows = F.cross_entropy(logits.double(), targets, ignore_index=-100, reduction="none").numpy()
    want_mean = F.cross_entropy(logits.double(), targets, ignore_index=-100, reduction="mean").item()
    assert np.allclose(loss, want_rows, rtol=1e-12, atol=1e-13)
    assert mean == pytest.approx(want_mean, rel=1e-12)


@pytest.mark.parametrize("kind", synth.ADVERSARIAL_KINDS)
def test_adversarial_rows_finite_and_consistent(kind):
    import torch.nn.functional as F
    x, hot = synth.adversarial_rows(kind, 10, 515, seed=90)
    xb = synth.to_bits(x)
    sm = oracle.softmax(xb)
    assert np.all(np.isfinite(sm)) and np.all(np.abs(sm.sum(axis=1) - 1) < 1e-12)
    assert np.allclose(sm, F.softmax(x.double(), dim=-1).numpy(), rtol=1e-12, atol=1e-300)
    w = synth.to_bits(torch.ones(515, dtype=torch.bfloat16))
    rn = oracle.rmsnorm(xb, w, 1e-6)
    assert np.all(np.isfinite(rn))
    assert np.allclose(rn, F.rms_norm(x.double(), (515,), None, float(np.float32(1e-6))).numpy(),
                       rtol=1e-12, atol=1e-300)
    t = hot.numpy().copy()
    t[1::2] = (t[1::2] + 1) % 515
    loss, mean, n = oracle.xent(xb, t)
    assert np.all(np.isfinite(loss)) and np.all(loss >= 0.0) and math.isfinite(mean)
    want = F.cross_entropy(x.double(), torch.from_numpy(t), reduction="none").numpy()
    assert np.allclose(loss, want, rtol=1e-12, atol=1e-13)


def test_thread_count_does_not_change_results():
    x = synth.softmax_inputs(64, 257, seed=5)
    xb = synth.to_bits(x)
    n0 = oracle.set_threads(0)
    oracle.set_threads(1)
    a = oracle.softmax(xb)
    oracle.set_threads(max(2, n0))
    b = oracle.softmax(xb)
    oracle.set_threads(n0)
    assert np.array_equal(a, b)

"""GPU parity for LayerNorm forward and the row-sum reduce: every CUDA path against the fp64
CPU checker, element by element, on the same seeded bf16 bit patterns, through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_bf16_close, bf16_tensor_to_f64, guarded
from test_gpu_parity import SHAPES, _legal_paths

pytestmark = pytest.mark.gpu
DEV = "cuda"
EPS = 1e-5


def _assert_ln_close(y, ref, x_bits, g_bits, b_bits, what):
    """The benchmark's bar (1.6e-2 * max(1, |ref|)) plus a one-rounding bound.  The output is
    z * gamma + beta, which may cancel, so the second bound is relative to |z * gamma| + |beta|
    rather than to |ref|: one bf16 rounding of the result plus fp32 evaluation error."""
    assert_bf16_close(y, ref, what, tight=False)
    got = bf16_tensor_to_f64(y).reshape(ref.shape)
    fin = np.isfinite(ref)
    beta = np.broadcast_to(oracle.bf16_to_f64(b_bits)[None, :], ref.shape)
    scale = np.abs(ref - beta) + np.abs(beta)
    bound = (2.0 ** -8 * 1.02) * np.abs(ref) + 4e-6 * scale + 2e-6   # 2e-6: fp32 error of the mean
    err = np.abs(got - ref)
    worst = float(np.max(err[fin] / bound[fin])) if fin.any() else 0.0
    assert worst <= 1.0, f"{what}: exceeds one-rounding bound by {worst:.3f}x"


@pytest.mark.parametrize("rows,D", SHAPES)
def test_layernorm_parity_all_paths(rows, D):
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(6, rows * 131 + D))
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    ref = oracle.layernorm(xb, gb, bb, EPS)
    xd, gd, bd = x.to(DEV), g.to(DEV), b.to(DEV)
    outs = {}
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_layernorm_fwd(xd, gd, bd, y, eps=EPS, path=path)
        torch.cuda.synchronize()
        check()
        _assert_ln_close(y, ref, xb, gb, bb, f"layernorm {rows}x{D} path {path}")
        outs[path] = y.clone()
    auto = ak.ak_layernorm_choose_path(rows, D, True)
    assert torch.equal(outs[ak.AK_PATH_AUTO].view(torch.int16), outs[auto].view(torch.int16))


@pytest.mark.parametrize("kind", synth.ADVERSARIAL_KINDS)
@pytest.mark.parametrize("D", [512, 4096, 4099])
def test_layernorm_adversarial_rows(kind, D):
    rows = 20
    x, _ = synth.adversarial_rows(kind, rows, D, synth.case_seed(7, D))
    _, g, b = synth.layernorm_inputs(1, D, 56)
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    ref = oracle.layernorm(xb, gb, bb, EPS)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y = ak.ak_layernorm_fwd(x.to(DEV), g.to(DEV), b.to(DEV), eps=EPS, path=path)
        assert torch.isfinite(y.float()).all()
        _assert_ln_close(y, ref, xb, gb, bb, f"layernorm adversarial {kind} D={D} path {path}")
        if kind in ("big_equal", "all_equal"):
            # a constant row has zero deviation: the output is beta, bit for bit
            assert torch.equal(y.view(torch.int16).cpu(), b.view(torch.int16)[None, :].expand(rows, D))


def test_layernorm_large_offset_small_spread():
    # mean far above the spread: values 1024 + {0, 8, 16, 24} (exact in bf16); a sum of squares
    # minus squared mean in fp32 would lose the variance, the centred passes must not
    D, rows = 4096, 16
    gen = torch.Generator().manual_seed(77)
    x = (1024.0 + 8.0 * torch.randint(0, 4, (rows, D), generator=gen)).to(torch.bfloat16)
    _, g, b = synth.layernorm_inputs(1, D, 57)
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    ref = oracle.layernorm(xb, gb, bb, EPS)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y = ak.ak_layernorm_fwd(x.to(DEV), g.to(DEV), b.to(DEV), eps=EPS, path=path)
        _assert_ln_close(y, ref, xb, gb, bb, f"layernorm offset 1024 path {path}")


def test_layernorm_ieee_conventions():
    # inf or NaN anywhere in a row makes the whole row NaN (inf - inf), as the definition does
    D = 1024
    x, g, b = synth.layernorm_inputs(4, D, 58)
    x[0, 5] = float("inf")
    x[1, 0] = float("-inf")
    x[2, 777] = float("nan")
    ref = oracle.layernorm(synth.to_bits(x), synth.to_bits(g), synth.to_bits(b), EPS)
    assert np.isnan(ref[:3]).all() and np.isfinite(ref[3]).all()
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y = ak.ak_layernorm_fwd(x.to(DEV), g.to(DEV), b.to(DEV), eps=EPS, path=path)
        assert_bf16_close(y, ref, f"layernorm inf/nan path {path}", tight=False)


def test_layernorm_misaligned_base_pointers():
    rows = 9
    for D in (1024, 1537):
        x, g, b = synth.layernorm_inputs(rows, D, 191)
        xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
        ref = oracle.layernorm(xb, gb, bb, EPS)
        for xo, yo, go, bo in ((1, 1, 0, 0), (1, 3, 0, 0), (0, 0, 5, 0), (0, 0, 0, 3), (2, 2, 2, 2),
                               (7, 7, 6, 4), (5, 5, 0, 2), (3, 3, 1, 1), (0, 0, 0, 0)):
            xbuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
            ybuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
            gbuf = torch.zeros(D + 8, dtype=torch.bfloat16, device=DEV)
            bbuf = torch.zeros(D + 8, dtype=torch.bfloat16, device=DEV)
            xv = xbuf[xo:xo + rows * D].view(rows, D)
            yv = ybuf[yo:yo + rows * D].view(rows, D)
            gv, bv = gbuf[go:go + D], bbuf[bo:bo + D]
            xv.copy_(x)
            gv.copy_(g)
            bv.copy_(b)
            ak.ak_layernorm_fwd(xv, gv, bv, yv, eps=EPS)
            torch.cuda.synchronize()
            _assert_ln_close(yv, ref, xb, gb, bb, f"layernorm D={D} offsets {xo},{yo},{go},{bo}")
            assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())


@pytest.mark.parametrize("rows,D,xo,few", [(1024, 1027, 0, 1000), (1500, 4001, 0, 1000), (1100, 2051, 3, 1000),
                                           (1500, 4099, 0, 200), (1024, 8190, 1, 200), (1030, 16379, 0, 255),
                                           (1025, 32754, 5, 250), (256, 32771, 0, 200), (300, 40001, 3, 255),
                                           (260, 65539, 1, 100)])
def test_layernorm_unaligned_rows_with_the_shift_table(rows, D, xo, few):
    """From 1024 rows on (256 for rows staged in shared memory: D of about 4090 and more), unaligned rows read gamma and beta
    from a table of all eight shifts written by a small kernel in front.  Parity on such launches,
    and the same bits as the launch without the table (fewer rows) gives for the rows they share."""
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(8, rows + D))
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    ref = oracle.layernorm(xb, gb, bb, EPS)
    xbuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
    ybuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
    xv = xbuf[xo:xo + rows * D].view(rows, D)
    yv = ybuf[xo:xo + rows * D].view(rows, D)
    xv.copy_(x)
    gd, bd = g.to(DEV), b.to(DEV)
    n0 = ak.ak_launch_count()
    ak.ak_layernorm_fwd(xv, gd, bd, yv, eps=EPS)
    torch.cuda.synchronize()
    assert ak.ak_launch_count() - n0 == 2          # the table kernel and the row kernel
    _assert_ln_close(yv, ref, xb, gb, bb, f"layernorm {rows}x{D} offset {xo} (shift table)")
    assert bool((ybuf[:xo] == 0).all()) and bool((ybuf[xo + rows * D:] == 0).all())
    y2buf = torch.zeros(few * D + 8, dtype=torch.bfloat16, device=DEV)
    y2 = y2buf[xo:xo + few * D].view(few, D)
    n0 = ak.ak_launch_count()
    ak.ak_layernorm_fwd(xv[:few], gd, bd, y2, eps=EPS)
    torch.cuda.synchronize()
    assert ak.ak_launch_count() - n0 == 1
    assert torch.equal(y2.view(torch.int16), yv[:few].view(torch.int16))
    # new parameters at the same addresses: the next launch must not see the old table
    gd.mul_(-0.5)
    bd.add_(1.0)
    ref2 = oracle.layernorm(xb, synth.to_bits(gd.cpu()), synth.to_bits(bd.cpu()), EPS)
    ak.ak_layernorm_fwd(xv, gd, bd, yv, eps=EPS)
    torch.cuda.synchronize()
    _assert_ln_close(yv, ref2, xb, synth.to_bits(gd.cpu()), synth.to_bits(bd.cpu()),
                     f"layernorm {rows}x{D} offset {xo} (shift table, new parameters)")


@pytest.mark.parametrize("rows,D", [(72, 4096), (72, 8192), (70, 32768), (72, 65536), (80, 40000), (66, 131080),
                                    (65, 128256), (70, 262144), (68, 36872), (66, 8190), (66, 65539), (65, 100001)])
def test_layernorm_far_shift_constant_and_offset_rows(rows, D):
    """The one-sweep moments are shifted by the mean of the row's first 16 bytes.  Every fourth
    row here has a huge first entry, so that shift lands far from the mean and the second sweep
    (shifted by the first mean estimate) runs; others are constant (output exactly beta) or sit at
    an offset of 1024 with a spread of 8.  More than 64 rows, so long rows take the many-row
    cluster layouts; every path that accepts the shape is run."""
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(23, rows * 131 + D))
    x[1::4, 0] = 65024.0
    x[2::8] = 3.5
    x[3::8] = (1024.0 + 8.0 * torch.randint(0, 4, x[3::8].shape, generator=torch.Generator().manual_seed(5))).to(x.dtype)
    xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
    ref = oracle.layernorm(xb, gb, bb, EPS)
    xd, gd, bd = x.to(DEV), g.to(DEV), b.to(DEV)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_layernorm_fwd(xd, gd, bd, y, eps=EPS, path=path)
        torch.cuda.synchronize()
        check()
        _assert_ln_close(y, ref, xb, gb, bb, f"layernorm {rows}x{D} path {path}")
        # a constant row has zero deviation: the output is beta, bit for bit
        assert torch.equal(y[2::8].view(torch.int16).cpu(), b.view(torch.int16)[None, :].expand(len(range(2, rows, 8)), D))
    assert ak.ak_wait_timeouts() == 0


def test_layernorm_in_place_and_empty():
    for D, paths in ((512, _legal_paths(512)), (4096, _legal_paths(4096)), (4099, _legal_paths(4099)),
                     (16384, _legal_paths(16384)), (131072, _legal_paths(131072))):
        x, g, b = synth.layernorm_inputs(11, D, 194)
        xb, gb, bb = synth.to_bits(x), synth.to_bits(g), synth.to_bits(b)
        ref = oracle.layernorm(xb, gb, bb, EPS)
        for path in paths:
            xd = x.to(DEV)
            ak.ak_layernorm_fwd(xd, g.to(DEV), b.to(DEV), xd, eps=EPS, path=path)
            _assert_ln_close(xd, ref, xb, gb, bb, f"in-place layernorm D={D} path {path}")
    e = torch.empty((0, 64), dtype=torch.bfloat16, device=DEV)
    w = torch.ones(64, dtype=torch.bfloat16, device=DEV)
    assert ak.ak_layernorm_fwd(e, w, w).shape == (0, 64)
    assert ak.ak_rowsum_fwd(e).shape == (0,)


def test_layernorm_rowsum_bitwise_determinism():
    x, g, b = synth.layernorm_inputs(4096, 4096, 196)
    xl, _, _ = synth.layernorm_inputs(64, 65536, 197)
    x9, g9, b9 = synth.layernorm_inputs(300, 4099, 198)
    xd, gd, bd, xld, x9d, g9d, b9d = (t.to(DEV) for t in (x, g, b, xl, x9, g9, b9))
    gl = torch.ones(65536, dtype=torch.bfloat16, device=DEV)
    first = None
    for _ in range(3):
        outs = [ak.ak_layernorm_fwd(xd, gd, bd).view(torch.int16).clone(),
                ak.ak_layernorm_fwd(xld, gl, gl).view(torch.int16).clone(),
                ak.ak_layernorm_fwd(x9d, g9d, b9d).view(torch.int16).clone(),
                ak.ak_rowsum_fwd(xd).view(torch.int32).clone(),
                ak.ak_rowsum_fwd(xld).view(torch.int32).clone(),
                ak.ak_rowsum_fwd(x9d).view(torch.int32).clone()]
        torch.empty(64 << 20, dtype=torch.uint8, device=DEV).fill_(1)
        torch.cuda.synchronize()
        if first is None:
            first = outs
        else:
            for a, c in zip(first, outs):
                assert torch.equal(a, c)


# ------------------------------------------------------------------------------ row sum
def _assert_rowsum_close(out, x_bits, what, rel=1e-6):
    ref = oracle.rowsum(x_bits)
    mag = np.abs(oracle.bf16_to_f64(x_bits)).sum(axis=1)
    got = out.detach().cpu().double().numpy()
    nan_ref = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan_ref), f"{what}: NaN pattern differs"
    fin = np.isfinite(ref)
    assert np.array_equal(got[~fin & ~nan_ref], ref[~fin & ~nan_ref]), f"{what}: inf differs"
    # fp32 accumulation in a fixed tree plus the final fp32 rounding of the result
    bound = rel * mag + 2.0 ** -24 * np.abs(ref) + 1e-45
    err = np.abs(got - ref)
    worst = float(np.max(err[fin] / bound[fin])) if fin.any() else 0.0
    assert worst <= 1.0, f"{what}: max err/bound = {worst:.3f}"


@pytest.mark.parametrize("rows,D", SHAPES + [(1000, 128), (300, 1025), (2, 262144)])
def test_rowsum_parity(rows, D):
    x, _, _ = synth.layernorm_inputs(rows, D, synth.case_seed(8, rows * 131 + D))
    out, check = guarded((rows,), torch.float32, DEV)
    ak.ak_rowsum_fwd(x.to(DEV), out)
    torch.cuda.synchronize()
    check()
    _assert_rowsum_close(out, synth.to_bits(x), f"rowsum {rows}x{D}")


@pytest.mark.parametrize("D", [1, 7, 8, 9, 100, 1000, 1024, 1025, 4099, 16392, 20000])
def test_rowsum_small_integers_are_exact_at_every_alignment(D):
    # integer entries in [-8, 8]: every fp32 partial sum is exact, so the result equals the
    # checker's bit for bit whatever the summation tree; offsets exercise head/tail handling
    rows = 13
    gen = torch.Generator().manual_seed(D)
    x = torch.randint(-8, 9, (rows, D), generator=gen).to(torch.bfloat16)
    ref = oracle.rowsum(synth.to_bits(x))
    for off in range(8):
        buf = torch.full((rows * D + 16,), 3.0, dtype=torch.bfloat16, device=DEV)  # poison around
        xv = buf[off:off + rows * D].view(rows, D)
        xv.copy_(x)
        out = ak.ak_rowsum_fwd(xv)
        assert np.array_equal(out.cpu().double().numpy(), ref), f"rowsum D={D} offset {off}"


@pytest.mark.parametrize("kind", synth.ADVERSARIAL_KINDS)
@pytest.mark.parametrize("D", [512, 4099, 32768])
def test_rowsum_adversarial(kind, D):
    x, _ = synth.adversarial_rows(kind, 20, D, synth.case_seed(9, D))
    out = ak.ak_rowsum_fwd(x.to(DEV))
    _assert_rowsum_close(out, synth.to_bits(x), f"rowsum adversarial {kind} D={D}", rel=1e-5)


def test_rowsum_ieee_conventions():
    x, _, _ = synth.layernorm_inputs(4, 4099, 59)
    x[0, 5] = float("inf")
    x[1, 4098] = float("-inf")
    x[2, 0] = float("nan")
    x[3, 1] = float("inf")
    x[3, 2] = float("-inf")
    out = ak.ak_rowsum_fwd(x.to(DEV)).cpu().numpy()
    assert out[0] == np.inf and out[1] == -np.inf and np.isnan(out[2]) and np.isnan(out[3])


@pytest.mark.parametrize("rows,D", [(1, 1 << 24), (1, (1 << 22) + 3), (4, 262144 + 5), (100, 65536), (591, 16384),
                                    (592, 16384), (1, 16383), (1, 16384)])
def test_rowsum_few_long_rows_and_vector_sum(rows, D):
    # a handful of long rows (a vector sum is rows == 1) take the split layout: partial sums by
    # many CTAs, then a fixed-order second launch
    x, _, _ = synth.layernorm_inputs(rows, D, synth.case_seed(22, rows + D), device=DEV)
    out, check = guarded((rows,), torch.float32, DEV)
    ak.ak_rowsum_fwd(x, out)
    again = ak.ak_rowsum_fwd(x)
    torch.cuda.synchronize()
    check()
    assert torch.equal(out.view(torch.int32), again.view(torch.int32))
    xb = synth.to_bits(x)
    _assert_rowsum_close(out, xb, f"rowsum split {rows}x{D}")
    # small integers: exact whatever the tree and the slicing, also from an odd base offset
    gen = torch.Generator().manual_seed(D)
    xi = torch.randint(-4, 5, (rows, D), generator=gen).to(torch.bfloat16)
    ref = oracle.rowsum(synth.to_bits(xi))
    for off in (0, 3):
        buf = torch.full((rows * D + 16,), 3.0, dtype=torch.bfloat16, device=DEV)
        xv = buf[off:off + rows * D].view(rows, D)
        xv.copy_(xi)
        assert np.array_equal(ak.ak_rowsum_fwd(xv).cpu().double().numpy(), ref), f"offset {off}"

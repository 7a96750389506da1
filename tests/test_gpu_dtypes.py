"""GPU parity of the fp16 and fp32 variants of RMSNorm, softmax and cross-entropy (the paper's
harness sweeps FP16 / BF16 / FP32): every path against the fp64 CPU checker on the same bits."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_close_dt, assert_loss_close, guarded
from test_gpu_parity import SHAPES, XENT_SHAPES

pytestmark = pytest.mark.gpu
DEV = "cuda"
DTS = [torch.float16, torch.float32]
NAME = synth.DTYPE_NAMES


def _legal_paths(D, dtype):
    nbytes = D * torch.empty((), dtype=dtype).element_size()
    paths = [ak.AK_PATH_GENERIC]
    if nbytes % 16 == 0 and nbytes >= 32 and nbytes <= 8 * 224 * 1024:
        paths.append(ak.AK_PATH_CLUSTER)
    if nbytes % 16 == 0 and nbytes <= 224 * 1024:
        paths.append(ak.AK_PATH_SMEM)
    if nbytes % 16 == 0 and nbytes <= 65536:
        paths.append(ak.AK_PATH_CTA)
    if nbytes % 16 == 0 and nbytes <= 4096:
        paths.append(ak.AK_PATH_WARP)
    return paths


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", SHAPES + [(5, 4), (7, 12), (9, 1028), (3, 57344)])
def test_rmsnorm_dt_parity_all_paths(rows, D, dtype):
    x, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(12, rows * 131 + D), dtype=dtype)
    ref = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 1e-6, NAME[dtype])
    xd, wd = x.to(DEV), w.to(DEV)
    outs = {}
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y, check = guarded((rows, D), dtype, DEV)
        ak.ak_rmsnorm_fwd_dt(xd, wd, y, eps=1e-6, path=path)
        torch.cuda.synchronize()
        check()
        assert_close_dt(y, ref, f"rmsnorm {NAME[dtype]} {rows}x{D} path {path}")
        outs[path] = y.clone()
    auto = ak.ak_choose_path_dt("rmsnorm", rows, D, dtype)
    assert torch.equal(outs[ak.AK_PATH_AUTO].view(torch.uint8), outs[auto].view(torch.uint8))


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", SHAPES + [(5, 4), (7, 12), (9, 1028), (3, 57344)])
def test_softmax_dt_parity_all_paths(rows, D, dtype):
    x = synth.softmax_inputs(rows, D, synth.case_seed(13, rows * 131 + D), mask_frac=0.3, dtype=dtype)
    ref = oracle.softmax_dt(synth.to_elems(x), NAME[dtype])
    xd = x.to(DEV)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y, check = guarded((rows, D), dtype, DEV)
        ak.ak_softmax_fwd_dt(xd, y, path=path)
        torch.cuda.synchronize()
        check()
        assert_close_dt(y, ref, f"softmax {NAME[dtype]} {rows}x{D} path {path}")
        assert bool((y[xd == float("-inf")] == 0).all()), "-inf entries must give exactly 0"
        assert bool(((y.float().sum(dim=-1) - 1).abs() <= 2e-3).all())


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", [(66, 65544), (65, 131080), (68, 36872), (66, 65539), (65, 100001)])
def test_softmax_rmsnorm_dt_many_long_rows(rows, D, dtype):
    """More than 64 long rows in fp16 / fp32: the many-row shapes of the cluster kernels (for the
    16-bit types the softmax kernel keeps some exponentials in registers and evaluates one pair in
    four of the others by a polynomial) and, unaligned, the staged kernels; ragged slices, a -inf
    half and a constant row."""
    x = synth.softmax_inputs(rows, D, synth.case_seed(33, rows * 131 + D), mask_frac=0.0, dtype=dtype)
    x[1, : D // 2] = float("-inf")
    x[2] = -7.5
    x[3, D - 1] = 60000.0
    ref = oracle.softmax_dt(synth.to_elems(x), NAME[dtype])
    xd = x.to(DEV)
    y, check = guarded((rows, D), dtype, DEV)
    ak.ak_softmax_fwd_dt(xd, y)
    torch.cuda.synchronize()
    check()
    assert_close_dt(y, ref, f"softmax {NAME[dtype]} {rows}x{D}")
    assert bool((y[xd == float("-inf")] == 0).all()), "-inf entries must give exactly 0"
    xr = torch.nan_to_num(x, neginf=-3.0)
    _, w = synth.rmsnorm_inputs(1, D, 81, dtype=dtype)
    refr = oracle.rmsnorm_dt(synth.to_elems(xr), synth.to_elems(w), 1e-6, NAME[dtype])
    y, check = guarded((rows, D), dtype, DEV)
    ak.ak_rmsnorm_fwd_dt(xr.to(DEV), w.to(DEV), y, eps=1e-6)
    torch.cuda.synchronize()
    check()
    assert_close_dt(y, refr, f"rmsnorm {NAME[dtype]} {rows}x{D}")
    assert ak.ak_wait_timeouts() == 0


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,V", XENT_SHAPES)
def test_xent_dt_parity_row_and_split(rows, V, dtype):
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(14, rows * 131 + V), dtype=dtype)
    ref_rows, ref_mean, n = oracle.xent_dt(synth.to_elems(lg), tg.numpy(), NAME[dtype])
    ld, td = lg.to(DEV), tg.to(DEV)
    variants = [(ak.AK_XENT_AUTO, 0), (ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 2), (ak.AK_XENT_SPLIT, 3),
                (ak.AK_XENT_SPLIT, 7)]
    for path, ns in variants:
        loss, mean = ak.ak_xent_fwd_dt(ld, td, path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert_loss_close(loss, ref_rows, f"xent {NAME[dtype]} {rows}x{V} path {path}/{ns}")
        assert bool((loss[td == -100] == 0).all())
        if n > 0:
            assert_loss_close(mean, np.array([ref_mean]), f"xent mean {NAME[dtype]} {rows}x{V}")


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("kind", synth.ADVERSARIAL_KINDS)
@pytest.mark.parametrize("D", [512, 4096, 4099])
def test_adversarial_rows_dt(kind, D, dtype):
    rows = 20
    xb, hot = synth.adversarial_rows(kind, rows, D, synth.case_seed(15, D))
    x = xb.to(dtype)   # 65024 is exact in fp16; 1e-30 becomes 0 there
    xe = synth.to_elems(x)
    xd = x.to(DEV)
    _, w = synth.rmsnorm_inputs(1, D, 155, dtype=dtype)
    ref = oracle.rmsnorm_dt(xe, synth.to_elems(w), 1e-6, NAME[dtype])
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y = ak.ak_rmsnorm_fwd_dt(xd, w.to(DEV), eps=1e-6, path=path)
        assert torch.isfinite(y.float()).all()
        assert_close_dt(y, ref, f"rmsnorm {NAME[dtype]} adversarial {kind} D={D} path {path}")
    ref = oracle.softmax_dt(xe, NAME[dtype])
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y = ak.ak_softmax_fwd_dt(xd, path=path)
        assert torch.isfinite(y.float()).all()
        assert_close_dt(y, ref, f"softmax {NAME[dtype]} adversarial {kind} D={D} path {path}")
    t = hot.clone()
    t[1::2] = (t[1::2] + 1) % D
    ref_rows, ref_mean, _ = oracle.xent_dt(xe, t.numpy(), NAME[dtype])
    for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 2), (ak.AK_XENT_SPLIT, 5)):
        loss, mean = ak.ak_xent_fwd_dt(xd, t.to(DEV), path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert torch.isfinite(loss).all() and bool((loss >= 0).all())
        assert_loss_close(loss, ref_rows, f"xent {NAME[dtype]} adversarial {kind} V={D} path {path}/{ns}")
        assert_loss_close(mean, np.array([ref_mean]), f"xent mean {NAME[dtype]} adversarial {kind}")


def test_fp16_range_edges():
    # subnormal inputs, the largest finite value, and an output that overflows fp16 to +inf
    D = 1024
    x = torch.zeros((4, D), dtype=torch.float16)
    x[0] = 2.0 ** -24                                   # all subnormal
    x[1, ::2] = 65504.0
    x[2, 0] = 65504.0                                   # rms = 65504/32: y[2,0] = 32 * w
    x[3] = torch.randn(D).to(torch.float16)
    w = torch.full((D,), 1.0, dtype=torch.float16)
    w[0] = 4096.0                                       # 32 * 4096 = 131072 > 65504: +inf in fp16
    ref = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 0.0, "f16")
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, torch.float16):
        y = ak.ak_rmsnorm_fwd_dt(x.to(DEV), w.to(DEV), eps=0.0, path=path)
        got = y.cpu().double().numpy()
        assert got[2, 0] == np.inf and abs(ref[2, 0] - 131072.0) < 1e-6
        ref_c = ref.copy()
        ref_c[2, 0] = np.inf                            # the type's own overflow
        assert_close_dt(y, ref_c, f"fp16 edges path {path}")
    refs = oracle.softmax_dt(synth.to_elems(x), "f16")
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, torch.float16):
        assert_close_dt(ak.ak_softmax_fwd_dt(x.to(DEV), path=path), refs, f"fp16 softmax edges path {path}")


@pytest.mark.parametrize("dtype", DTS)
def test_misaligned_base_pointers_dt(dtype):
    D, rows = 1024, 9
    x, w = synth.rmsnorm_inputs(rows, D, 291, dtype=dtype)
    ref = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 1e-6, NAME[dtype])
    per16 = 16 // x.element_size()
    for xo, yo, wo in ((1, 1, 0), (1, 3, 0), (0, 0, 1), (3, 0, 1), (2, 2, 2), (per16 - 1, per16 - 1, per16 - 2)):
        xbuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        ybuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        wbuf = torch.zeros(D + 8, dtype=dtype, device=DEV)
        xv, yv, wv = xbuf[xo:xo + rows * D].view(rows, D), ybuf[yo:yo + rows * D].view(rows, D), wbuf[wo:wo + D]
        xv.copy_(x)
        wv.copy_(w)
        ak.ak_rmsnorm_fwd_dt(xv, wv, yv, eps=1e-6)
        torch.cuda.synchronize()
        assert_close_dt(yv, ref, f"rmsnorm {NAME[dtype]} offsets {xo},{yo},{wo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())
    xs = synth.softmax_inputs(rows, D, 292, dtype=dtype)
    ref = oracle.softmax_dt(synth.to_elems(xs), NAME[dtype])
    for xo, yo in ((1, 1), (3, 2)):
        xbuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        ybuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        xv, yv = xbuf[xo:xo + rows * D].view(rows, D), ybuf[yo:yo + rows * D].view(rows, D)
        xv.copy_(xs)
        ak.ak_softmax_fwd_dt(xv, yv)
        torch.cuda.synchronize()
        assert_close_dt(yv, ref, f"softmax {NAME[dtype]} offsets {xo},{yo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())
    lg, tg = synth.xent_inputs(rows, 1000, 293, dtype=dtype)
    ref_rows, _, _ = oracle.xent_dt(synth.to_elems(lg), tg.numpy(), NAME[dtype])
    for off in (1, 3):
        lbuf = torch.zeros(rows * 1000 + 8, dtype=dtype, device=DEV)
        lv = lbuf[off:off + rows * 1000].view(rows, 1000)
        lv.copy_(lg)
        for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 3)):
            loss, _ = ak.ak_xent_fwd_dt(lv, tg.to(DEV), path=path, nsplit=ns)
            torch.cuda.synchronize()
            assert_loss_close(loss, ref_rows, f"xent {NAME[dtype]} offset {off}")


@pytest.mark.parametrize("dtype", DTS)
def test_in_place_and_determinism_dt(dtype):
    for D in (512, 4096, 4099):
        x, w = synth.rmsnorm_inputs(11, D, 294, dtype=dtype)
        ref = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 1e-6, NAME[dtype])
        xs = synth.softmax_inputs(11, D, 295, dtype=dtype)
        refs = oracle.softmax_dt(synth.to_elems(xs), NAME[dtype])
        for path in _legal_paths(D, dtype):
            xd = x.to(DEV)
            ak.ak_rmsnorm_fwd_dt(xd, w.to(DEV), xd, eps=1e-6, path=path)
            assert_close_dt(xd, ref, f"in-place rmsnorm {NAME[dtype]} D={D} path {path}")
            xd = xs.to(DEV)
            ak.ak_softmax_fwd_dt(xd, xd, path=path)
            assert_close_dt(xd, refs, f"in-place softmax {NAME[dtype]} D={D} path {path}")
    x, w = synth.rmsnorm_inputs(2048, 4096, 296, device=DEV, dtype=dtype)
    xs = synth.softmax_inputs(1024, 8192, 297, device=DEV, dtype=dtype)
    lg, tg = synth.xent_inputs(256, 32000, 298, device=DEV, dtype=dtype)
    first = None
    for _ in range(3):
        outs = [ak.ak_rmsnorm_fwd_dt(x, w).view(torch.uint8).clone(), ak.ak_softmax_fwd_dt(xs).view(torch.uint8).clone()]
        for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 4)):
            loss, mean = ak.ak_xent_fwd_dt(lg, tg, path=path, nsplit=ns)
            outs += [loss.view(torch.int32).clone(), mean.view(torch.int32).clone()]
        torch.empty(64 << 20, dtype=torch.uint8, device=DEV).fill_(1)
        torch.cuda.synchronize()
        if first is None:
            first = outs
        else:
            for a, b in zip(first, outs):
                assert torch.equal(a, b)


def test_bf16_through_the_dt_entry_points_is_bit_identical():
    x, w = synth.rmsnorm_inputs(300, 4096, 299, device=DEV)
    assert torch.equal(ak.ak_rmsnorm_fwd(x, w).view(torch.int16), ak.ak_rmsnorm_fwd_dt(x, w).view(torch.int16))
    xs = synth.softmax_inputs(300, 8192, 300, device=DEV)
    assert torch.equal(ak.ak_softmax_fwd(xs).view(torch.int16), ak.ak_softmax_fwd_dt(xs).view(torch.int16))
    lg, tg = synth.xent_inputs(64, 32000, 301, device=DEV)
    a, am = ak.ak_xent_fwd(lg, tg)
    b, bm = ak.ak_xent_fwd_dt(lg, tg)
    assert torch.equal(a.view(torch.int32), b.view(torch.int32)) and torch.equal(am.view(torch.int32), bm.view(torch.int32))


# ------------------------------------------------------------------ LayerNorm and row-sum in fp16 / fp32
def _assert_ln_close_dt(y, ref, b, what):
    """Main bar of the element type, plus one rounding relative to |z * gamma| + |beta| (the
    output may cancel) and the fp32 error of the mean."""
    assert_close_dt(y, ref, what, tight=False)
    got = y.detach().cpu().double().numpy().reshape(ref.shape)
    beta = np.broadcast_to(b.double().numpy()[None, :], ref.shape)
    rnd = {torch.float16: 2.0 ** -11 * 1.02, torch.float32: 2.0 ** -23}[y.dtype]
    bound = rnd * np.abs(ref) + 4e-6 * (np.abs(ref - beta) + np.abs(beta)) + 2e-6
    fin = np.isfinite(ref)
    worst = float(np.max(np.abs(got - ref)[fin] / bound[fin])) if fin.any() else 0.0
    assert worst <= 1.0, f"{what}: exceeds one-rounding bound by {worst:.3f}x"


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", SHAPES + [(5, 4), (7, 12), (9, 1028), (3, 57344)])
def test_layernorm_dt_parity_all_paths(rows, D, dtype):
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(19, rows * 131 + D), dtype=dtype)
    ref = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, NAME[dtype])
    xd, gd, bd = x.to(DEV), g.to(DEV), b.to(DEV)
    outs = {}
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y, check = guarded((rows, D), dtype, DEV)
        ak.ak_layernorm_fwd_dt(xd, gd, bd, y, eps=1e-5, path=path)
        torch.cuda.synchronize()
        check()
        _assert_ln_close_dt(y, ref, b, f"layernorm {NAME[dtype]} {rows}x{D} path {path}")
        outs[path] = y.clone()
    auto = ak.ak_choose_path_dt("layernorm", rows, D, dtype)
    assert torch.equal(outs[ak.AK_PATH_AUTO].view(torch.uint8), outs[auto].view(torch.uint8))


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", [(72, 1024), (72, 4096), (70, 16384), (72, 65536), (66, 40008), (65, 131076), (66, 4099)])
def test_layernorm_dt_far_shift_constant_and_offset_rows(rows, D, dtype):
    """fp16 / fp32 counterpart of the bf16 test of the same name: rows whose first entry is an
    outlier (the shift of the moments lands far from the mean, so the second sweep runs), constant
    rows (output exactly beta) and rows at an offset of 1024 with a spread of 8, on every path."""
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(29, rows * 131 + D), dtype=dtype)
    x[1::4, 0] = 60000.0
    x[2::8] = 3.5
    x[3::8] = (1024.0 + 8.0 * torch.randint(0, 4, x[3::8].shape, generator=torch.Generator().manual_seed(5))).to(dtype)
    ref = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, NAME[dtype])
    xd, gd, bd = x.to(DEV), g.to(DEV), b.to(DEV)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
        y, check = guarded((rows, D), dtype, DEV)
        ak.ak_layernorm_fwd_dt(xd, gd, bd, y, eps=1e-5, path=path)
        torch.cuda.synchronize()
        check()
        _assert_ln_close_dt(y, ref, b, f"layernorm {NAME[dtype]} {rows}x{D} path {path}")
        assert torch.equal(y[2::8].cpu(), b[None, :].expand(len(range(2, rows, 8)), D))
    assert ak.ak_wait_timeouts() == 0


@pytest.mark.parametrize("dtype", DTS)
@pytest.mark.parametrize("rows,D", SHAPES + [(1000, 128), (300, 1025), (5, 4), (7, 13)])
def test_rowsum_dt_parity_and_exact_integers(rows, D, dtype):
    x, _, _ = synth.layernorm_inputs(rows, D, synth.case_seed(20, rows * 131 + D), dtype=dtype)
    out, check = guarded((rows,), torch.float32, DEV)
    ak.ak_rowsum_fwd_dt(x.to(DEV), out)
    torch.cuda.synchronize()
    check()
    ref = oracle.rowsum_dt(synth.to_elems(x), NAME[dtype])
    mag = x.double().abs().sum(dim=-1).numpy()
    err = np.abs(out.cpu().double().numpy() - ref)
    assert float(np.max(err / (1e-6 * mag + 2.0 ** -24 * np.abs(ref) + 1e-45))) <= 1.0
    # integer entries: every fp32 partial sum is exact whatever the tree, at every base offset
    gen = torch.Generator().manual_seed(D)
    xi = torch.randint(-8, 9, (min(rows, 13), D), generator=gen).to(dtype)
    refi = oracle.rowsum_dt(synth.to_elems(xi), NAME[dtype])
    per16 = 16 // xi.element_size()
    for off in range(per16):
        buf = torch.full((xi.numel() + 16,), 3.0, dtype=dtype, device=DEV)
        xv = buf[off:off + xi.numel()].view(xi.shape)
        xv.copy_(xi)
        assert np.array_equal(ak.ak_rowsum_fwd_dt(xv).cpu().double().numpy(), refi), f"offset {off}"


@pytest.mark.parametrize("dtype", DTS)
def test_layernorm_dt_adversarial_misaligned_in_place(dtype):
    for kind in synth.ADVERSARIAL_KINDS:
        for D in (512, 4099):
            xb, _ = synth.adversarial_rows(kind, 20, D, synth.case_seed(21, D))
            x = xb.to(dtype)
            _, g, b = synth.layernorm_inputs(1, D, 156, dtype=dtype)
            ref = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, NAME[dtype])
            for path in [ak.AK_PATH_AUTO] + _legal_paths(D, dtype):
                y = ak.ak_layernorm_fwd_dt(x.to(DEV), g.to(DEV), b.to(DEV), eps=1e-5, path=path)
                assert torch.isfinite(y.float()).all()
                _assert_ln_close_dt(y, ref, b, f"layernorm {NAME[dtype]} adversarial {kind} D={D} path {path}")
                if kind in ("big_equal", "all_equal"):
                    assert torch.equal(y.cpu(), b[None, :].expand(20, D))     # constant rows give beta exactly
    rows, D = 9, 1537
    x, g, b = synth.layernorm_inputs(rows, D, 391, dtype=dtype)
    ref = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, NAME[dtype])
    per16 = 16 // x.element_size()
    for xo, yo, go, bo in ((1, 1, 0, 0), (1, 3, 0, 0), (0, 0, 1, 0), (2, 2, 2, 2), (per16 - 1, per16 - 1, 2, 0), (0, 0, 0, 0)):
        xbuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        ybuf = torch.zeros(rows * D + 8, dtype=dtype, device=DEV)
        gbuf = torch.zeros(D + 8, dtype=dtype, device=DEV)
        bbuf = torch.zeros(D + 8, dtype=dtype, device=DEV)
        xv, yv = xbuf[xo:xo + rows * D].view(rows, D), ybuf[yo:yo + rows * D].view(rows, D)
        gv, bv = gbuf[go:go + D], bbuf[bo:bo + D]
        xv.copy_(x); gv.copy_(g); bv.copy_(b)
        ak.ak_layernorm_fwd_dt(xv, gv, bv, yv, eps=1e-5)
        torch.cuda.synchronize()
        _assert_ln_close_dt(yv, ref, b, f"layernorm {NAME[dtype]} offsets {xo},{yo},{go},{bo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())
    xd = x.to(DEV)
    ak.ak_layernorm_fwd_dt(xd, g.to(DEV), b.to(DEV), xd, eps=1e-5)
    _assert_ln_close_dt(xd, ref, b, f"layernorm {NAME[dtype]} in place")


def test_layernorm_fp16_unaligned_rows_with_the_shift_table():
    rows, D = 1200, 2051
    x, g, b = synth.layernorm_inputs(rows, D, 393, dtype=torch.float16)
    ref = oracle.layernorm_dt(synth.to_elems(x), synth.to_elems(g), synth.to_elems(b), 1e-5, "f16")
    n0 = ak.ak_launch_count()
    y = ak.ak_layernorm_fwd_dt(x.to(DEV), g.to(DEV), b.to(DEV), eps=1e-5)
    torch.cuda.synchronize()
    assert ak.ak_launch_count() - n0 == 2
    _assert_ln_close_dt(y, ref, b, "layernorm f16 1200x2051 (shift table)")


def test_layernorm_rowsum_bf16_through_the_dt_entry_points_is_bit_identical():
    x, g, b = synth.layernorm_inputs(300, 4096, 392, device=DEV)
    assert torch.equal(ak.ak_layernorm_fwd(x, g, b).view(torch.int16), ak.ak_layernorm_fwd_dt(x, g, b).view(torch.int16))
    assert torch.equal(ak.ak_rowsum_fwd(x).view(torch.int32), ak.ak_rowsum_fwd_dt(x).view(torch.int32))

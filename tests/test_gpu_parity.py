"""GPU parity: every CUDA path against the fp64 CPU checker, element by element, on the
same seeded bf16 bit patterns, through the C ABI (ctypes binding)."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_bf16_close, assert_loss_close, guarded

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _needs_clusters():
    """Tests of what the dispatcher sends to thread-block clusters do not apply when the library's
    diagnostic switch AK_DISABLE_CLUSTERS keeps every row on one CTA."""
    if os.environ.get("AK_DISABLE_CLUSTERS", "0") not in ("", "0"):
        pytest.skip("the cluster layouts are switched off in this environment")


WARP, CTA, GEN, SMEM = ak.AK_PATH_WARP, ak.AK_PATH_CTA, ak.AK_PATH_GENERIC, ak.AK_PATH_SMEM
CLUSTER = ak.AK_PATH_CLUSTER


def _legal_paths(D):
    paths = [GEN]
    if D % 8 == 0 and D >= 16 and D * 2 <= 8 * 224 * 1024:
        paths.append(CLUSTER)
    if D % 8 == 0 and D * 2 <= 224 * 1024:
        paths.append(SMEM)
    if D % 8 == 0 and D <= 32768:
        paths.append(CTA)
    if D % 8 == 0 and D <= 2048:
        paths.append(WARP)
    return paths


# shapes: several tiles plus ragged tails, every vectors-per-thread count of both register
# paths, non-multiples of 8, the paper's edge sizes (1023, 1537, 4097) and the benchmark's
# (4099); rows chosen so the checker stays fast
SHAPES = [(256, 1024), (1, 8), (3, 16), (37, 64), (129, 256), (65, 512), (33, 776), (40, 1000),
          (33, 1280), (19, 1536), (21, 1792), (64, 2048), (17, 4096), (1, 4096), (23, 3072),
          (9, 5120), (16, 8192), (7, 11008), (12, 16384), (5, 20480), (3, 24576), (3, 28672),
          (6, 32768), (3, 65536), (2, 114688), (5, 1), (4, 7), (31, 1023), (11, 1537), (9, 4097), (13, 4099), (2, 40000),
          (3, 128257),
          # unaligned rows in the registers of 256- and 512-thread CTAs, and just past them
          (10, 8190), (6, 10247), (5, 12290), (4, 16379), (3, 24571), (3, 32754), (2, 32771)]


@pytest.mark.parametrize("rows,D", SHAPES)
def test_rmsnorm_parity_all_paths(rows, D):
    seed = 0 if (rows, D) == (256, 1024) else synth.case_seed(2, rows * 131 + D)
    x, w = synth.rmsnorm_inputs(rows, D, seed)
    ref = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
    xd, wd = x.to(DEV), w.to(DEV)
    outs = {}
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_rmsnorm_fwd(xd, wd, y, eps=1e-6, path=path)
        torch.cuda.synchronize()
        check()
        assert_bf16_close(y, ref, f"rmsnorm {rows}x{D} path {path}")
        outs[path] = y.clone()
    auto = ak.ak_rmsnorm_choose_path(rows, D, True)
    assert torch.equal(outs[ak.AK_PATH_AUTO].view(torch.int16), outs[auto].view(torch.int16))


@pytest.mark.parametrize("rows,D", SHAPES)
def test_softmax_parity_all_paths(rows, D):
    x = synth.softmax_inputs(rows, D, synth.case_seed(3, rows * 131 + D), mask_frac=0.3)
    ref = oracle.softmax(synth.to_bits(x))
    xd = x.to(DEV)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_softmax_fwd(xd, y, path=path)
        torch.cuda.synchronize()
        check()
        assert_bf16_close(y, ref, f"softmax {rows}x{D} path {path}")
        neg_inf = (xd.view(torch.int16) == -128)  # 0xFF80
        assert bool((y[neg_inf].view(torch.int16) == 0).all()), "-inf entries must give exactly +0"
        sums = y.float().sum(dim=-1)
        assert bool(((sums - 1).abs() <= 4e-3 + 2e-3).all())


XENT_SHAPES = [(4, 8), (64, 1000), (33, 4099), (5, 1), (7, 9), (40, 8192), (24, 32000),
               (12, 50304), (8, 128256), (6, 128257), (300, 2048)]


@pytest.mark.parametrize("rows,V", XENT_SHAPES)
def test_xent_parity_row_and_split(rows, V):
    logits, targets = synth.xent_inputs(rows, V, synth.case_seed(4, rows * 131 + V), ignore_frac=0.2)
    ref_rows, ref_mean, n = oracle.xent(synth.to_bits(logits), targets.numpy())
    ld, td = logits.to(DEV), targets.to(DEV)
    variants = [(ak.AK_XENT_AUTO, 0), (ak.AK_XENT_ROW, 0)]
    variants += [(ak.AK_XENT_SPLIT, ns) for ns in (1, 2, 3, 7, 64)]
    for path, ns in variants:
        loss, check = guarded((rows,), torch.float32, DEV)
        mean, check_mean = guarded((1,), torch.float32, DEV)
        ak.ak_xent_fwd(ld, td, -100, loss, mean, path=path, nsplit=ns)
        torch.cuda.synchronize()
        check()
        check_mean()
        assert_loss_close(loss, ref_rows, f"xent rows {rows}x{V} path {path}/{ns}")
        assert_loss_close(mean, np.array([ref_mean]), f"xent mean {rows}x{V} path {path}/{ns}")
        ign = td == -100
        assert bool((loss[ign] == 0).all())
        assert bool((loss[~ign] >= 0).all())
    # caller-provided workspace variant gives the same bits as the allocating entry point
    nbytes = ak.ak_xent_workspace_bytes(rows, V)
    ws = torch.empty((max(nbytes, 8),), dtype=torch.uint8, device=DEV)
    l1, m1 = ak.ak_xent_fwd(ld, td)
    l2, m2 = ak.ak_xent_fwd_ws(ld, td, ws if nbytes else None)
    torch.cuda.synchronize()
    assert torch.equal(l1.view(torch.int32), l2.view(torch.int32))
    assert torch.equal(m1.view(torch.int32), m2.view(torch.int32)) or (torch.isnan(m1).all() and torch.isnan(m2).all())


@pytest.mark.parametrize("V", [1000, 32000])
def test_xent_masked_vocabulary_and_extreme_gaps(V):
    """-inf logits (a masked vocabulary) contribute nothing, a -inf target gives +inf, gaps far
    beyond the polynomial's clamp (2^-125) and rows dominated by one element stay accurate."""
    rows = 24
    logits, targets = synth.xent_inputs(rows, V, synth.case_seed(5, V), ignore_frac=0.0)
    g = torch.Generator().manual_seed(V)
    masked = torch.rand((rows, V), generator=g) < 0.3
    logits = logits.masked_fill(masked, float("-inf"))
    logits[3, :] = -200.0                      # everything 200 below ...
    logits[3, 17] = 50.0                       # ... one element: loss 0 on it, 250 elsewhere
    logits[4, :] = torch.where(torch.arange(V) % 2 == 0, 0.0, -120.0).to(torch.bfloat16)
    targets[3] = 17
    targets[5] = int(torch.nonzero(masked[5])[0])          # target on a -inf logit -> +inf
    ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(logits), targets.numpy())
    assert np.isinf(ref_rows[5]) and ref_rows[3] == 0.0
    for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 3)):
        loss, mean = ak.ak_xent_fwd(logits.to(DEV), targets.to(DEV), path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert_loss_close(loss, ref_rows, f"masked vocabulary V={V} path {path}")
        assert torch.isinf(mean).all() and np.isinf(ref_mean)


def test_xent_mean_skipped_when_null():
    logits, targets = synth.xent_inputs(16, 512, 7)
    loss, mean = ak.ak_xent_fwd(logits.to(DEV), targets.to(DEV), want_mean=False)
    torch.cuda.synchronize()
    assert mean is None and loss.shape == (16,)


def test_xent_conventions_bad_targets_and_all_ignored():
    logits, _ = synth.xent_inputs(6, 40, 8)
    ld = logits.to(DEV)
    t = torch.tensor([0, 40, -1, -100, 39, 5], dtype=torch.int64)
    ref_rows, ref_mean, n = oracle.xent(synth.to_bits(logits), t.numpy())
    for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 3)):
        loss, mean = ak.ak_xent_fwd(ld, t.to(DEV), path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert_loss_close(loss, ref_rows, "bad targets")
        assert torch.isnan(mean).all() and np.isnan(ref_mean)
        t_ign = torch.full((6,), -100, dtype=torch.int64, device=DEV)
        loss, mean = ak.ak_xent_fwd(ld, t_ign, path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert bool((loss == 0).all()) and torch.isnan(mean).all()
        # a custom ignore_index
        t7 = torch.tensor([7, 1, 7, 2, 3, 7], dtype=torch.int64)
        r7, m7, _ = oracle.xent(synth.to_bits(logits), t7.numpy(), ignore_index=7)
        loss, mean = ak.ak_xent_fwd(ld, t7.to(DEV), ignore_index=7, path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert_loss_close(loss, r7, "ignore_index=7")
        assert_loss_close(mean, np.array([m7]), "ignore_index=7 mean")
    # NaN planted in an ignored row must not leak; rows = 0 gives NaN mean
    l2 = logits.clone()
    l2[3, 4] = float("nan")
    loss, mean = ak.ak_xent_fwd(l2.to(DEV), torch.tensor([0, 1, 2, -100, 4, 5], device=DEV))
    torch.cuda.synchronize()
    assert torch.isfinite(loss).all() and torch.isfinite(mean).all()
    empty = torch.empty((0, 40), dtype=torch.bfloat16, device=DEV)
    loss, mean = ak.ak_xent_fwd(empty, torch.empty((0,), dtype=torch.int64, device=DEV))
    torch.cuda.synchronize()
    assert loss.numel() == 0 and torch.isnan(mean).all()


def test_softmax_ieee_conventions():
    x = torch.zeros((4, 24), dtype=torch.bfloat16)
    x[0, :] = float("-inf")           # fully masked row -> NaN
    x[1, 3] = float("inf")            # +inf -> NaN row
    x[2, 5] = float("nan")            # NaN -> NaN row
    x[3, :] = torch.arange(24) * 0.25  # ordinary row
    ref = oracle.softmax(synth.to_bits(x))
    for path in (WARP, CTA, GEN, SMEM, CLUSTER):
        y = ak.ak_softmax_fwd(x.to(DEV), path=path)
        torch.cuda.synchronize()
        assert_bf16_close(y, ref, f"softmax conventions path {path}")


@pytest.mark.parametrize("D", [65544, 131072, 128257, 1048576])
def test_ieee_conventions_on_rows_split_over_clusters(D):
    """The same conventions where a row is spread over several CTAs (staged slices, aligned and
    not, and streamed slices): a NaN, a +inf or a fully masked row in ONE slice decides the whole
    row; RMSNorm and LayerNorm rows with an inf or NaN element come out as the checker says."""
    x = synth.softmax_inputs(5, D, synth.case_seed(17, D), mask_frac=0.0)
    x[0, :] = float("-inf")                    # fully masked row -> NaN
    x[1, D - 3] = float("inf")                 # +inf in the last slice -> NaN row
    x[2, 5] = float("nan")                     # NaN in the first slice -> NaN row
    x[3, D // 2:] = float("-inf")              # whole slices masked: exact zeros there
    ref = oracle.softmax(synth.to_bits(x))
    y = ak.ak_softmax_fwd(x.to(DEV))
    torch.cuda.synchronize()
    assert_bf16_close(y, ref, f"softmax conventions D={D}")
    assert bool((y[3, D // 2:].view(torch.int16) == 0).all())
    xn, w = synth.rmsnorm_inputs(4, D, synth.case_seed(18, D))
    _, g, b = synth.layernorm_inputs(1, D, 81)
    xn[1, D - 2] = float("inf")
    xn[2, 7] = float("nan")
    yr = ak.ak_rmsnorm_fwd(xn.to(DEV), w.to(DEV))
    yl = ak.ak_layernorm_fwd(xn.to(DEV), g.to(DEV), b.to(DEV))
    torch.cuda.synchronize()
    assert_bf16_close(yr, oracle.rmsnorm(synth.to_bits(xn), synth.to_bits(w), 1e-6), f"rmsnorm conventions D={D}")
    assert_bf16_close(yl, oracle.layernorm(synth.to_bits(xn), synth.to_bits(g), synth.to_bits(b), 1e-5),
                      f"layernorm conventions D={D}", tight=False)


@pytest.mark.parametrize("kind", synth.ADVERSARIAL_KINDS)
@pytest.mark.parametrize("D", [512, 4096, 4099])
def test_adversarial_rows_all_ops(kind, D):
    rows = 20
    x, hot = synth.adversarial_rows(kind, rows, D, synth.case_seed(5, D))
    xb = synth.to_bits(x)
    xd = x.to(DEV)
    _, w = synth.rmsnorm_inputs(1, D, 55)
    ref = oracle.rmsnorm(xb, synth.to_bits(w), 1e-6)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y = ak.ak_rmsnorm_fwd(xd, w.to(DEV), eps=1e-6, path=path)
        assert torch.isfinite(y.float()).all()
        assert_bf16_close(y, ref, f"rmsnorm adversarial {kind} D={D} path {path}")
    ref = oracle.softmax(xb)
    for path in [ak.AK_PATH_AUTO] + _legal_paths(D):
        y = ak.ak_softmax_fwd(xd, path=path)
        assert torch.isfinite(y.float()).all()
        assert_bf16_close(y, ref, f"softmax adversarial {kind} D={D} path {path}")
    t = hot.clone()
    t[1::2] = (t[1::2] + 1) % D       # half of the rows aim beside the planted logit
    ref_rows, ref_mean, _ = oracle.xent(xb, t.numpy())
    for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 2), (ak.AK_XENT_SPLIT, 5)):
        loss, mean = ak.ak_xent_fwd(xd, t.to(DEV), path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert torch.isfinite(loss).all() and torch.isfinite(mean).all()
        assert bool((loss >= 0).all())
        assert_loss_close(loss, ref_rows, f"xent adversarial {kind} V={D} path {path}/{ns}")
        assert_loss_close(mean, np.array([ref_mean]), f"xent adversarial mean {kind} V={D}")


def test_all_equal_softmax_4099_prints_two_to_minus_12():
    # 1/4099 rounds to 2^-12 in bf16, so an all-equal row of length 4099 is 2^-12 everywhere
    x = torch.full((2, 4099), 3.0, dtype=torch.bfloat16, device=DEV)
    y = ak.ak_softmax_fwd(x)
    assert bool((y.float() == 2.0 ** -12).all())


def test_misaligned_base_pointers_take_generic_path():
    D, rows = 1024, 9
    x, w = synth.rmsnorm_inputs(rows, D, 91)
    ref = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
    for xo, yo, wo in ((1, 1, 0), (1, 3, 0), (0, 0, 5), (3, 0, 1), (2, 2, 2), (7, 7, 6), (5, 5, 0)):
        xbuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
        ybuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
        wbuf = torch.zeros(D + 8, dtype=torch.bfloat16, device=DEV)
        xv = xbuf[xo:xo + rows * D].view(rows, D)
        yv = ybuf[yo:yo + rows * D].view(rows, D)
        wv = wbuf[wo:wo + D]
        xv.copy_(x)
        wv.copy_(w)
        ak.ak_rmsnorm_fwd(xv, wv, yv, eps=1e-6)
        torch.cuda.synchronize()
        assert_bf16_close(yv, ref, f"rmsnorm offsets {xo},{yo},{wo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())
    xs = synth.softmax_inputs(rows, D, 92)
    ref = oracle.softmax(synth.to_bits(xs))
    for xo, yo in ((1, 1), (5, 2)):
        xbuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
        ybuf = torch.zeros(rows * D + 8, dtype=torch.bfloat16, device=DEV)
        xv = xbuf[xo:xo + rows * D].view(rows, D)
        yv = ybuf[yo:yo + rows * D].view(rows, D)
        xv.copy_(xs)
        ak.ak_softmax_fwd(xv, yv)
        torch.cuda.synchronize()
        assert_bf16_close(yv, ref, f"softmax offsets {xo},{yo}")
        assert bool((ybuf[:yo] == 0).all()) and bool((ybuf[yo + rows * D:] == 0).all())
    logits, targets = synth.xent_inputs(rows, 1000, 93)
    ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(logits), targets.numpy())
    lbuf = torch.zeros(rows * 1000 + 8, dtype=torch.bfloat16, device=DEV)
    lv = lbuf[3:3 + rows * 1000].view(rows, 1000)
    lv.copy_(logits)
    for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 3)):
        loss, mean = ak.ak_xent_fwd(lv, targets.to(DEV), path=path, nsplit=ns)
        torch.cuda.synchronize()
        assert_loss_close(loss, ref_rows, "xent offset 3")


def test_in_place_is_allowed():
    for D, paths in ((512, (WARP, CTA, GEN, SMEM, CLUSTER)), (4096, (CTA, GEN, SMEM, CLUSTER)), (4099, (GEN,)),
                     (16384, (CTA, SMEM, CLUSTER)), (131072, (CLUSTER,))):
        x, w = synth.rmsnorm_inputs(11, D, 94)
        ref = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
        xs = synth.softmax_inputs(11, D, 95)
        refs = oracle.softmax(synth.to_bits(xs))
        for path in paths:
            xd = x.to(DEV)
            ak.ak_rmsnorm_fwd(xd, w.to(DEV), xd, eps=1e-6, path=path)
            assert_bf16_close(xd, ref, f"in-place rmsnorm D={D} path {path}")
            xd = xs.to(DEV)
            ak.ak_softmax_fwd(xd, xd, path=path)
            assert_bf16_close(xd, refs, f"in-place softmax D={D} path {path}")


def test_bitwise_determinism_three_runs():
    x, w = synth.rmsnorm_inputs(4096, 4096, 96)
    xs = synth.softmax_inputs(2048, 8192, 97)
    logits, targets = synth.xent_inputs(512, 32000, 98)
    xd, wd, xsd, ld, td = x.to(DEV), w.to(DEV), xs.to(DEV), logits.to(DEV), targets.to(DEV)
    first = None
    for _ in range(3):
        outs = [ak.ak_rmsnorm_fwd(xd, wd).view(torch.int16).clone(),
                ak.ak_softmax_fwd(xsd).view(torch.int16).clone()]
        for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 4)):
            loss, mean = ak.ak_xent_fwd(ld, td, path=path, nsplit=ns)
            outs += [loss.view(torch.int32).clone(), mean.view(torch.int32).clone()]
        # disturb the machine between runs
        torch.empty(64 << 20, dtype=torch.uint8, device=DEV).fill_(1)
        torch.cuda.synchronize()
        if first is None:
            first = outs
        else:
            for a, b in zip(first, outs):
                assert torch.equal(a, b)


_DIGEST_SNIPPET = r"""
import hashlib, sys, torch
sys.path.insert(0, sys.argv[1])
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
h = hashlib.sha256()
x, w = synth.rmsnorm_inputs(1024, 4096, 196)
h.update(ak.ak_rmsnorm_fwd(x.cuda(), w.cuda()).cpu().view(torch.int16).numpy().tobytes())
xs = synth.softmax_inputs(512, 16384, 197)
h.update(ak.ak_softmax_fwd(xs.cuda()).cpu().view(torch.int16).numpy().tobytes())
x9, w9 = synth.rmsnorm_inputs(300, 4099, 199)
h.update(ak.ak_rmsnorm_fwd(x9.cuda(), w9.cuda()).cpu().view(torch.int16).numpy().tobytes())
lg, tg = synth.xent_inputs(256, 50304, 198)
for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 5)):
    loss, mean = ak.ak_xent_fwd(lg.cuda(), tg.cuda(), path=path, nsplit=ns)
    h.update(loss.cpu().numpy().tobytes()); h.update(mean.cpu().numpy().tobytes())
print(h.hexdigest())
"""


def test_bitwise_determinism_across_processes():
    """Two fresh processes produce byte-identical outputs (register, shared-memory, staged and
    both cross-entropy layouts)."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    digests = [subprocess.run([sys.executable, "-c", _DIGEST_SNIPPET, root], capture_output=True, text=True,
                              check=True).stdout.strip() for _ in range(2)]
    assert len(digests[0]) == 64 and digests[0] == digests[1]


def test_host_buffer_variants_match_device_path():
    x, w = synth.rmsnorm_inputs(5000, 4096, 101)       # > one 16 MiB chunk, ragged last chunk
    y_dev = ak.ak_rmsnorm_fwd(x.to(DEV), w.to(DEV)).cpu()
    xh, yh = x.pin_memory(), torch.empty_like(x).pin_memory()
    ak.ak_rmsnorm_fwd_host(xh, w, yh)
    assert torch.equal(yh.view(torch.int16), y_dev.view(torch.int16))
    xs = synth.softmax_inputs(3000, 8192, 102)
    y_dev = ak.ak_softmax_fwd(xs.to(DEV)).cpu()
    yh = torch.empty_like(xs)
    ak.ak_softmax_fwd_host(xs, yh)                     # pageable memory works too
    assert torch.equal(yh.view(torch.int16), y_dev.view(torch.int16))
    logits, targets = synth.xent_inputs(700, 32000, 103)
    ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(logits), targets.numpy())
    loss_h = torch.empty(700, dtype=torch.float32)
    mean_h = torch.empty(1, dtype=torch.float32)
    ak.ak_xent_fwd_host(logits.pin_memory(), targets, loss_h, mean_h)
    assert_loss_close(loss_h, ref_rows, "host xent rows")
    assert_loss_close(mean_h, np.array([ref_mean]), "host xent mean")
    ak.lib().ak_host_arena_release()


def test_non_default_stream_and_launch_counter():
    x, w = synth.rmsnorm_inputs(64, 2048, 104)
    ref = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
    s = torch.cuda.Stream()
    xd, wd = x.to(DEV), w.to(DEV)
    torch.cuda.synchronize()
    before = ak.ak_launch_count()
    with torch.cuda.stream(s):
        y = ak.ak_rmsnorm_fwd(xd, wd)
    s.synchronize()
    assert ak.ak_launch_count() == before + 1
    assert_bf16_close(y, ref, "non-default stream")


@pytest.mark.parametrize("rows,D", [(1, 16), (3, 24), (5, 4104), (64, 16384), (65, 16384), (7, 131072), (2, 458752),
                                    (1, 917504), (3, 128256), (9, 65544)])
def test_cluster_path_slices_and_limits(rows, D):
    """Rows split over a thread-block cluster: slices of unequal length (D / 8 not a multiple of
    the cluster size), the shortest legal rows (two vectors), rows far beyond one CTA's shared
    memory up to the 8 x 224 KiB limit, and both sides of the few-rows rule.  All three ops, forced
    and as the dispatcher's own choice; -inf and identical-value rows included."""
    _needs_clusters()
    x, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(9, rows * 131 + D))
    if rows > 1:
        x[0, : D // 2] = float("-inf")      # whole slices of -inf (softmax); replaced by -3 for the norms
    xs = x.clone()
    xr = torch.nan_to_num(x, neginf=-3.0)
    _, g, b = synth.layernorm_inputs(1, D, 77)
    ref_r = oracle.rmsnorm(synth.to_bits(xr), synth.to_bits(w), 1e-6)
    ref_s = oracle.softmax(synth.to_bits(xs))
    ref_l = oracle.layernorm(synth.to_bits(xr), synth.to_bits(g), synth.to_bits(b), 1e-5)
    for path in (CLUSTER, ak.AK_PATH_AUTO):
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_rmsnorm_fwd(xr.to(DEV), w.to(DEV), y, eps=1e-6, path=path)
        torch.cuda.synchronize()
        check()
        assert_bf16_close(y, ref_r, f"rmsnorm cluster {rows}x{D} path {path}")
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_softmax_fwd(xs.to(DEV), y, path=path)
        torch.cuda.synchronize()
        check()
        assert_bf16_close(y, ref_s, f"softmax cluster {rows}x{D} path {path}")
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        ak.ak_layernorm_fwd(xr.to(DEV), g.to(DEV), b.to(DEV), y, eps=1e-5, path=path)
        torch.cuda.synchronize()
        check()
        # z * gamma + beta may cancel, so only the benchmark's bar applies here (the one-rounding
        # bound relative to |z * gamma| + |beta| is checked in the LayerNorm tests proper)
        assert_bf16_close(y, ref_l, f"layernorm cluster {rows}x{D} path {path}", tight=False)
    if D * 2 > 8 * 224 * 1024:
        return
    want = CLUSTER if (D * 2 > 65536 or (rows <= 64 and D * 2 >= 32768)) else None
    if want is not None:
        assert ak.ak_rmsnorm_choose_path(rows, D, True) == want
        assert ak.ak_softmax_choose_path(rows, D, True) == want


@pytest.mark.parametrize("rows,D", [(66, 65544), (70, 100000), (65, 131080), (68, 36872), (72, 262152),
                                    (66, 65539), (65, 100001), (67, 128257), (66, 50001)])
def test_many_long_rows_ragged_slices(rows, D):
    """More than 64 long rows take the many-row shapes of the cluster kernels (128-thread CTAs that
    keep exponentials in registers for softmax, one exchange for LayerNorm) and, unaligned, the
    staged or cluster-staged kernels from their per-op lengths on.  Ragged slices (the vectors of a
    row not a multiple of the cluster size, edge elements at both ends), rows with a -inf half, a
    constant row and a row with one huge entry; every op against the oracle on the dispatcher's
    own choice."""
    x, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(31, rows * 131 + D))
    x[1, : D // 2] = float("-inf")
    x[2] = -7.5
    x[3, D - 1] = 65024.0
    x[4, 0] = 65024.0
    # a ramp from 0 down to -110: its exponentials pass through the bottom of the fp32 range (e^-87.3 =
    # 2^-126), where the polynomial and the special-function evaluations flush differently
    x[5] = torch.linspace(0.0, -110.0, D).to(torch.bfloat16)
    xs = x.clone()
    xr = torch.nan_to_num(x, neginf=-3.0)
    _, g, b = synth.layernorm_inputs(1, D, 79)
    ref_r = oracle.rmsnorm(synth.to_bits(xr), synth.to_bits(w), 1e-6)
    ref_s = oracle.softmax(synth.to_bits(xs))
    ref_l = oracle.layernorm(synth.to_bits(xr), synth.to_bits(g), synth.to_bits(b), 1e-5)
    y, check = guarded((rows, D), torch.bfloat16, DEV)
    ak.ak_rmsnorm_fwd(xr.to(DEV), w.to(DEV), y, eps=1e-6)
    torch.cuda.synchronize()
    check()
    assert_bf16_close(y, ref_r, f"rmsnorm {rows}x{D}")
    y, check = guarded((rows, D), torch.bfloat16, DEV)
    ak.ak_softmax_fwd(xs.to(DEV), y)
    torch.cuda.synchronize()
    check()
    assert_bf16_close(y, ref_s, f"softmax {rows}x{D}")
    y, check = guarded((rows, D), torch.bfloat16, DEV)
    ak.ak_layernorm_fwd(xr.to(DEV), g.to(DEV), b.to(DEV), y, eps=1e-5)
    torch.cuda.synchronize()
    check()
    assert_bf16_close(y, ref_l, f"layernorm {rows}x{D}", tight=False)
    assert torch.equal(y[2].view(torch.int16).cpu(), b.view(torch.int16))   # constant row: beta exactly
    assert ak.ak_wait_timeouts() == 0


def test_cluster_path_rejects_rows_it_cannot_hold():
    x = torch.zeros((1, 8), dtype=torch.bfloat16, device=DEV)           # one vector: nothing to split
    w = torch.ones((8,), dtype=torch.bfloat16, device=DEV)
    with pytest.raises(ak.AkError):
        ak.ak_rmsnorm_fwd(x, w, path=CLUSTER)
    big = torch.zeros((1, 917512), dtype=torch.bfloat16, device=DEV)    # one vector beyond 8 x 224 KiB: streamed
    y = ak.ak_softmax_fwd(big)
    y2 = ak.ak_softmax_fwd(big, path=CLUSTER)
    torch.cuda.synchronize()
    v = y.float()
    assert bool((v == v[0, 0]).all()) and abs(float(v[0, 0]) * 917512 - 1.0) < 2.0 ** -8
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))


@pytest.mark.parametrize("rows,D", [(1, 917512), (3, 1048576), (2, 2000008), (70, 1000000)])
def test_rows_of_any_length_streamed_by_a_cluster(rows, D):
    """Aligned rows beyond the shared memory of eight CTAs: each CTA of the cluster streams its slice
    from global memory, partial results through the mailboxes.  All three ops, in place as well."""
    x, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(15, rows * 131 + D))
    _, g, b = synth.layernorm_inputs(1, D, 80)
    xs = synth.softmax_inputs(rows, D, synth.case_seed(16, rows * 131 + D), mask_frac=0.3)
    idx = sorted({0, rows - 1, rows // 2})
    for name, run, ref in (
            ("rmsnorm", lambda t, o: ak.ak_rmsnorm_fwd(t, w.to(DEV), o, eps=1e-6),
             oracle.rmsnorm(synth.to_bits(x[idx]), synth.to_bits(w), 1e-6)),
            ("layernorm", lambda t, o: ak.ak_layernorm_fwd(t, g.to(DEV), b.to(DEV), o, eps=1e-5),
             oracle.layernorm(synth.to_bits(x[idx]), synth.to_bits(g), synth.to_bits(b), 1e-5)),
            ("softmax", lambda t, o: ak.ak_softmax_fwd(t, o), oracle.softmax(synth.to_bits(xs[idx])))):
        src = (xs if name == "softmax" else x).to(DEV)
        y, check = guarded((rows, D), torch.bfloat16, DEV)
        run(src, y)
        torch.cuda.synchronize()
        check()
        assert_bf16_close(y[idx], ref, f"{name} {rows}x{D} (streamed)", tight=(name != "layernorm"))
        first = y.clone()
        run(src, src)                                                   # in place
        torch.cuda.synchronize()
        assert torch.equal(first.view(torch.int16), src.view(torch.int16))


@pytest.mark.parametrize("D", [1024, 2048, 4096, 8192])
def test_small_launches_fetch_parameters_early_with_the_same_bits(D):
    """Launches too small to fill the GPU request w (gamma, beta) together with the row instead of
    after the reductions; that changes when the loads are issued, not the arithmetic: the rows a
    small and a large launch share come out bit for bit the same."""
    big, small = 3000, 24
    x, w = synth.rmsnorm_inputs(big, D, synth.case_seed(11, D), device=DEV)
    _, g, b = synth.layernorm_inputs(1, D, 78, device=DEV)
    y_big = ak.ak_rmsnorm_fwd(x, w)
    y_small = ak.ak_rmsnorm_fwd(x[:small].contiguous(), w)
    l_big = ak.ak_layernorm_fwd(x, g, b)
    l_small = ak.ak_layernorm_fwd(x[:small].contiguous(), g, b)
    torch.cuda.synchronize()
    assert torch.equal(y_big[:small].view(torch.int16), y_small.view(torch.int16))
    assert torch.equal(l_big[:small].view(torch.int16), l_small.view(torch.int16))
    ref = oracle.rmsnorm(synth.to_bits(x[:small].cpu()), synth.to_bits(w.cpu()), 1e-6)
    assert_bf16_close(y_small, ref, f"rmsnorm {small}x{D} (early weights)")


@pytest.mark.parametrize("rows,D,xo", [(3, 128257, 0), (2, 300001, 3), (20, 20001, 0), (64, 16385, 5), (1, 917490, 1),
                                       (5, 114700, 7), (65, 114689, 0)])
def test_unaligned_rows_split_over_a_cluster(rows, D, xo):
    """Rows that are not 16-byte aligned and either too long for one CTA's shared memory or too few
    to fill the GPU: the covering vectors of the row's own phase are split over a thread-block
    cluster.  Guard bands around y; every row starts in a different phase."""
    x = synth.softmax_inputs(rows, D, synth.case_seed(12, rows * 131 + D), mask_frac=0.3)
    ref = oracle.softmax(synth.to_bits(x))
    xbuf = torch.zeros(rows * D + 16, dtype=torch.bfloat16, device=DEV)
    ybuf = torch.full((rows * D + 16,), 7.0, dtype=torch.bfloat16, device=DEV)
    xv = xbuf[xo:xo + rows * D].view(rows, D)
    yv = ybuf[xo:xo + rows * D].view(rows, D)
    xv.copy_(x)
    ak.ak_softmax_fwd(xv, yv)
    torch.cuda.synchronize()
    assert_bf16_close(yv, ref, f"softmax {rows}x{D} offset {xo}")
    assert bool((ybuf[:xo] == 7.0).all()) and bool((ybuf[xo + rows * D:] == 7.0).all())
    # RMSNorm and LayerNorm on the same layout (finite inputs)
    xn, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(13, rows * 131 + D))
    _, g, b = synth.layernorm_inputs(1, D, 79)
    xv.copy_(xn)
    ybuf.fill_(7.0)
    ak.ak_rmsnorm_fwd(xv, w.to(DEV), yv, eps=1e-6)
    torch.cuda.synchronize()
    assert_bf16_close(yv, oracle.rmsnorm(synth.to_bits(xn), synth.to_bits(w), 1e-6), f"rmsnorm {rows}x{D} offset {xo}")
    assert bool((ybuf[:xo] == 7.0).all()) and bool((ybuf[xo + rows * D:] == 7.0).all())
    ybuf.fill_(7.0)
    ak.ak_layernorm_fwd(xv, g.to(DEV), b.to(DEV), yv, eps=1e-5)
    torch.cuda.synchronize()
    assert_bf16_close(yv, oracle.layernorm(synth.to_bits(xn), synth.to_bits(g), synth.to_bits(b), 1e-5),
                      f"layernorm {rows}x{D} offset {xo}", tight=False)
    assert bool((ybuf[:xo] == 7.0).all()) and bool((ybuf[xo + rows * D:] == 7.0).all())


def test_layernorm_unaligned_cluster_with_the_shift_table():
    """Enough long unaligned rows for both the cluster layout and the table of shifted parameters
    (two launches: the table kernel, then the cluster kernel as its programmatic dependent)."""
    _needs_clusters()
    rows, D = 300, 114700
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(14, D), device=DEV)
    n0 = ak.ak_launch_count()
    y = ak.ak_layernorm_fwd(x, g, b, eps=1e-5)
    torch.cuda.synchronize()
    assert ak.ak_launch_count() - n0 == 2
    idx = [0, 1, 7, 150, 299]
    it = torch.tensor(idx, device=DEV)
    ref = oracle.layernorm(synth.to_bits(x[it].cpu()), synth.to_bits(g.cpu()), synth.to_bits(b.cpu()), 1e-5)
    assert_bf16_close(y[it], ref, "layernorm 300x114700 sampled rows (cluster + shift table)", tight=False)
    # the same rows without the table (fewer rows): same bits
    y2 = ak.ak_layernorm_fwd(x[:200].contiguous(), g, b, eps=1e-5)
    torch.cuda.synchronize()
    assert torch.equal(y2.view(torch.int16), y[:200].view(torch.int16))


def test_magnitudes_beyond_the_square_range_of_fp32_are_pinned():
    """bf16 holds magnitudes up to 3.4e38, but the norms add squares in fp32: once a row's sum
    of squares (RMSNorm) or of squared deviations (LayerNorm) passes 3.4e38 it becomes inf,
    1/sqrt(inf) is 0 and the row comes out as 0 (RMSNorm) or as beta (LayerNorm), where the fp64
    definition gives +-w and +-gamma + beta.  This is the documented behaviour (ak.h), stated
    here so that it cannot change unnoticed: exact zeros / beta, never NaN or garbage; rows just
    inside the range follow the definition; softmax and cross-entropy, which only subtract the
    maximum, follow the definition at any magnitude."""
    D = 1024
    sign = torch.tensor([1.0, -1.0]).repeat(D // 2)
    w = (1.0 + 0.25 * torch.arange(D) / D).to(torch.bfloat16)
    beta = (0.5 - torch.arange(D) / D).to(torch.bfloat16)
    for exp2, inside in ((70, False), (62, False), (50, True)):
        # D * (2^e)^2 = 2^(2e + 10): beyond fp32's 2^128 for e = 62 and 70, inside for e = 50
        x = (sign * 2.0 ** exp2).to(torch.bfloat16).repeat(3, 1)
        xb = synth.to_bits(x)
        ref_r = oracle.rmsnorm(xb, synth.to_bits(w), 1e-6)
        ref_l = oracle.layernorm(xb, synth.to_bits(w), synth.to_bits(beta), 1e-5)
        assert np.isfinite(ref_r).all() and np.isfinite(ref_l).all()       # the definition is finite
        for path in (ak.AK_PATH_AUTO, GEN, SMEM, CLUSTER):
            yr = ak.ak_rmsnorm_fwd(x.to(DEV), w.to(DEV), eps=1e-6, path=path)
            yl = ak.ak_layernorm_fwd(x.to(DEV), w.to(DEV), beta.to(DEV), eps=1e-5, path=path)
            torch.cuda.synchronize()
            if inside:
                assert_bf16_close(yr, ref_r, f"rmsnorm |x| = 2^{exp2} path {path}")
                assert_bf16_close(yl, ref_l, f"layernorm |x| = 2^{exp2} path {path}", tight=False)
            else:
                assert bool((yr.float() == 0).all()), f"rmsnorm |x| = 2^{exp2}: not exact (signed) zeros"
                assert torch.equal(yl.cpu().view(torch.int16), beta.repeat(3, 1).view(torch.int16)), \
                    f"layernorm |x| = 2^{exp2}: not beta"
        ys = ak.ak_softmax_fwd(x.to(DEV))
        assert_bf16_close(ys, oracle.softmax(xb), f"softmax |x| = 2^{exp2}")
        t = torch.tensor([0, 1, 2])
        loss, mean = ak.ak_xent_fwd(x.to(DEV), t.to(DEV))
        ref_rows, ref_mean, _ = oracle.xent(xb, t.numpy())
        assert_loss_close(loss, ref_rows, f"xent |x| = 2^{exp2}")
        assert_loss_close(mean, np.array([ref_mean]), f"xent mean |x| = 2^{exp2}")

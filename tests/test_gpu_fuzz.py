"""Seeded random shapes and base-pointer offsets for every op against the fp64 CPU checker:
small and odd row lengths, rows that straddle 16-byte boundaries in every phase, x and y in
equal and in different phases, guard bands around every output."""
import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_bf16_close, assert_close_dt, assert_loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAME = synth.DTYPE_NAMES


def _cases(seed, n):
    rng = np.random.default_rng(seed)
    out = []
    for i in range(n):
        rows = int(rng.integers(1, 24))
        kind = i % 5
        if kind == 4:
            # long rows: split over thread-block clusters when 16-byte aligned (up to 8 CTAs' shared
            # memory), staged or multi-pass when not
            rows = int(rng.integers(1, 5))
            D = 8 * int(rng.integers(2048, 40000)) + int(rng.choice([0, 0, 0, 0, 1, -1, 4]))
        elif kind == 0:
            D = int(rng.integers(1, 65))
        elif kind == 1:
            D = int(rng.integers(65, 2100))
        elif kind == 2:
            D = int(rng.integers(2100, 9000))
        else:
            D = int(rng.choice([8, 16, 1024, 4096, 8176, 8184, 8192, 8200, 16384])) + int(rng.integers(-1, 2))
        xo = int(rng.integers(0, 8))
        yo = xo if rng.random() < 0.7 else int(rng.integers(0, 8))
        wo = int(rng.integers(0, 8))
        out.append((rows, max(1, D), xo, yo, wo))
    return out


def _place(t, off, fill=0.0):
    """Copy t into a fresh device buffer at element offset `off`; returns (buffer, view)."""
    n = t.numel()
    buf = torch.full((n + 16,), fill, dtype=t.dtype, device=DEV)
    view = buf[off:off + n].view(t.shape)
    view.copy_(t)
    return buf, view


def _guards_untouched(buf, off, n, fill):
    return bool((buf[:off] == fill).all()) and bool((buf[off + n:] == fill).all())


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16])
def test_fuzz_rmsnorm_softmax(dtype):
    for rows, D, xo, yo, wo in _cases(101 if dtype == torch.bfloat16 else 102, 48):
        what = f"{NAME[dtype]} {rows}x{D} offsets x{xo} y{yo} w{wo}"
        x, w = synth.rmsnorm_inputs(rows, D, 1000 + rows * 7 + D, dtype=dtype)
        ref = oracle.rmsnorm_dt(synth.to_elems(x), synth.to_elems(w), 1e-6, NAME[dtype])
        _, xv = _place(x, xo)
        _, wv = _place(w, wo)
        ybuf = torch.full((rows * D + 16,), 7.0, dtype=dtype, device=DEV)
        yv = ybuf[yo:yo + rows * D].view(rows, D)
        ak.ak_rmsnorm_fwd_dt(xv, wv, yv)
        torch.cuda.synchronize()
        assert_close_dt(yv, ref, "rmsnorm " + what)
        assert _guards_untouched(ybuf, yo, rows * D, 7.0), "rmsnorm wrote outside y: " + what
        xs = synth.softmax_inputs(rows, D, 2000 + rows * 7 + D, mask_frac=0.3, dtype=dtype)
        ref = oracle.softmax_dt(synth.to_elems(xs), NAME[dtype])
        _, xv = _place(xs, xo)
        ybuf = torch.full((rows * D + 16,), 7.0, dtype=dtype, device=DEV)
        yv = ybuf[yo:yo + rows * D].view(rows, D)
        ak.ak_softmax_fwd_dt(xv, yv)
        torch.cuda.synchronize()
        assert_close_dt(yv, ref, "softmax " + what)
        assert _guards_untouched(ybuf, yo, rows * D, 7.0), "softmax wrote outside y: " + what


def test_fuzz_layernorm_rowsum():
    for rows, D, xo, yo, wo in _cases(103, 48):
        what = f"{rows}x{D} offsets x{xo} y{yo} g{wo}"
        x, g, b = synth.layernorm_inputs(rows, D, 3000 + rows * 7 + D)
        xb = synth.to_bits(x)
        ref = oracle.layernorm(xb, synth.to_bits(g), synth.to_bits(b), 1e-5)
        _, xv = _place(x, xo)
        _, gv = _place(g, wo)
        _, bv = _place(b, (wo * 3) % 8)
        ybuf = torch.full((rows * D + 16,), 7.0, dtype=torch.bfloat16, device=DEV)
        yv = ybuf[yo:yo + rows * D].view(rows, D)
        ak.ak_layernorm_fwd(xv, gv, bv, yv, eps=1e-5)
        torch.cuda.synchronize()
        if D > 1:   # D = 1 makes every deviation zero: 0 * rsqrt(eps) + beta, compared below
            assert_bf16_close(yv, ref, "layernorm " + what, tight=False)
        else:
            assert torch.equal(yv.view(torch.int16).cpu(), b.view(torch.int16)[None, :].expand(rows, 1))
        assert _guards_untouched(ybuf, yo, rows * D, 7.0), "layernorm wrote outside y: " + what
        s = ak.ak_rowsum_fwd(xv).cpu().double().numpy()
        mag = np.abs(oracle.bf16_to_f64(xb)).sum(axis=1)
        sref = oracle.rowsum(xb)
        assert np.all(np.abs(s - sref) <= 1e-6 * mag + 2.0 ** -24 * np.abs(sref)), "rowsum " + what


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_fuzz_xent(dtype):
    per16 = 16 // torch.empty((), dtype=dtype).element_size()
    for rows, V, xo, _, _ in _cases(104 if dtype == torch.bfloat16 else 105, 40):
        xo %= per16
        what = f"{NAME[dtype]} {rows}x{V} offset {xo}"
        lg, tg = synth.xent_inputs(rows, V, 4000 + rows * 7 + V, dtype=dtype, ignore_frac=0.15)
        ref_rows, ref_mean, n = oracle.xent_dt(synth.to_elems(lg), tg.numpy(), NAME[dtype])
        _, lv = _place(lg, xo)
        td = tg.to(DEV)
        for path, ns in ((ak.AK_XENT_ROW, 0), (ak.AK_XENT_SPLIT, 1 + rows % 5)):
            loss, mean = ak.ak_xent_fwd_dt(lv, td, path=path, nsplit=ns)
            torch.cuda.synchronize()
            assert_loss_close(loss, ref_rows, f"xent {what} path {path}/{ns}")
            if n > 0:
                assert_loss_close(mean, np.array([ref_mean]), f"xent mean {what}")
            else:
                assert bool(torch.isnan(mean).all())


def test_fuzz_rope():
    rng = np.random.default_rng(106)
    for i in range(30):
        n_seq, S = int(rng.integers(1, 9)), int(rng.integers(1, 40))
        Dh = 2 * int(rng.integers(1, 70)) if i % 2 else int(rng.choice([8, 32, 64, 96, 128, 256, 512]))
        dtype = [torch.bfloat16, torch.float16, torch.float32][i % 3]
        off = int(rng.integers(0, 4)) if i % 4 == 0 else 0
        pos = int(rng.integers(0, 100000))
        x = synth.rope_inputs(n_seq, S, Dh, 5000 + i, dtype=dtype)
        ref = oracle.rope(synth.to_elems(x), NAME[dtype], pos_offset=pos)
        _, xv = _place(x, off)
        ybuf = torch.full((x.numel() + 16,), 7.0, dtype=dtype, device=DEV)
        yv = ybuf[off:off + x.numel()].view(x.shape)
        ak.ak_rope_fwd(xv, yv, pos_offset=pos)
        torch.cuda.synchronize()
        assert_close_dt(yv, ref, f"rope {NAME[dtype]} {n_seq}x{S}x{Dh} off {off} pos {pos}", tight=False)
        assert _guards_untouched(ybuf, off, x.numel(), 7.0)


def test_two_streams_and_graph_replay():
    """Re-entrancy: the same ops enqueued on two streams at once (disjoint buffers) give the
    results of the serial calls; and a captured graph holding one call of every op replays to
    the same bits."""
    x, w = synth.rmsnorm_inputs(2048, 4096, 601, device=DEV)
    xs = synth.softmax_inputs(1024, 8192, 602, device=DEV)
    lg, tg = synth.xent_inputs(2048, 32000, 603, device=DEV)
    xl, g, b = synth.layernorm_inputs(2048, 4096, 604, device=DEV)
    xr = synth.rope_inputs(16, 512, 128, 605, device=DEV, dtype=torch.float16)
    # unaligned rows, enough of them for the shifted-parameter table (scratch + dependent launch)
    xu, gu, bu = synth.layernorm_inputs(1500, 2051, 606, device=DEV)
    # rows split over thread-block clusters (a few long rows; rows beyond one CTA's shared memory)
    xc = synth.softmax_inputs(8, 131072, 609, device=DEV)
    xk, wk = synth.rmsnorm_inputs(300, 128256, 610, device=DEV)

    def run_all(stream=None):
        loss, mean = ak.ak_xent_fwd(lg, tg, stream=stream)
        return [ak.ak_rmsnorm_fwd(x, w, stream=stream), ak.ak_softmax_fwd(xs, stream=stream), loss, mean,
                ak.ak_layernorm_fwd(xl, g, b, stream=stream), ak.ak_rowsum_fwd(xl, stream=stream),
                ak.ak_rope_fwd(xr, stream=stream), ak.ak_layernorm_fwd(xu, gu, bu, stream=stream),
                ak.ak_softmax_fwd(xc, stream=stream), ak.ak_rmsnorm_fwd(xk, wk, stream=stream)]

    serial = [t.clone() for t in run_all()]
    torch.cuda.synchronize()
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    with torch.cuda.stream(s1):
        a = run_all(s1)
    with torch.cuda.stream(s2):
        c = run_all(s2)
    torch.cuda.synchronize()
    for ref, u, v in zip(serial, a, c):
        assert torch.equal(ref.view(torch.uint8), u.view(torch.uint8))
        assert torch.equal(ref.view(torch.uint8), v.view(torch.uint8))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        run_all()                                   # warm-up outside the capture
        with torch.cuda.graph(graph, stream=side):
            outs = run_all()
    torch.cuda.current_stream().wait_stream(side)
    for _ in range(2):
        for t in outs:
            t.view(torch.uint8).zero_()
        graph.replay()
        torch.cuda.synchronize()
        for ref, u in zip(serial, outs):
            assert torch.equal(ref.view(torch.uint8), u.view(torch.uint8))


def test_first_call_inside_a_stream_capture():
    """A process whose very first library call happens inside a CUDA-graph capture (nothing
    warmed up, no scratch pool yet): the ops that take stream-ordered scratch capture, replay and
    match the eager results taken afterwards."""
    import subprocess
    import sys
    code = r"""
import torch
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
dev = "cuda"
xu, gu, bu = synth.layernorm_inputs(1500, 2051, 606, device=dev)
xl, _, _ = synth.layernorm_inputs(16, 65536, 607, device=dev)
lg, tg = synth.xent_inputs(16, 65536, 608, device=dev)
torch.cuda.synchronize()
side = torch.cuda.Stream()
side.wait_stream(torch.cuda.current_stream())
graph = torch.cuda.CUDAGraph()
with torch.cuda.stream(side):
    with torch.cuda.graph(graph, stream=side):
        loss, mean = ak.ak_xent_fwd(lg, tg)
        outs = [ak.ak_layernorm_fwd(xu, gu, bu), ak.ak_rowsum_fwd(xl), loss, mean]
torch.cuda.current_stream().wait_stream(side)
graph.replay()
torch.cuda.synchronize()
got = [t.clone() for t in outs]
loss, mean = ak.ak_xent_fwd(lg, tg)
eager = [ak.ak_layernorm_fwd(xu, gu, bu), ak.ak_rowsum_fwd(xl), loss, mean]
torch.cuda.synchronize()
for a, b in zip(got, eager):
    assert torch.equal(a.view(torch.uint8), b.view(torch.uint8))
print("capture-first ok")
"""
    import os
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    r = subprocess.run([sys.executable, "-c", code], cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "capture-first ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]


def test_clusters_switched_off_by_the_environment():
    """AK_DISABLE_CLUSTERS=1 keeps every row on one CTA (the layouts a device that cannot
    co-schedule clusters falls back to): same results within tolerance, long rows included."""
    import os
    import subprocess
    import sys
    code = r"""
import numpy as np, torch
import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
dev = "cuda"
def widen(t):
    bits = t.cpu().view(torch.int16).numpy().view(np.uint16)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
for rows, D in ((5, 16384), (3, 65536), (2, 131072), (3, 128257), (4, 40001)):
    assert ak.ak_softmax_choose_path(rows, D, True) != ak.AK_PATH_CLUSTER
    x, w = synth.rmsnorm_inputs(rows, D, 700 + D)
    y = ak.ak_rmsnorm_fwd(x.to(dev), w.to(dev))
    ref = oracle.rmsnorm(synth.to_bits(x), synth.to_bits(w), 1e-6)
    assert (np.abs(widen(y) - ref) / np.maximum(1.0, np.abs(ref))).max() <= 1.6e-2
    xs = synth.softmax_inputs(rows, D, 800 + D)
    ys = ak.ak_softmax_fwd(xs.to(dev))
    refs = oracle.softmax(synth.to_bits(xs))
    assert np.abs(widen(ys) - refs).max() <= 1.6e-2
    xl, g, b = synth.layernorm_inputs(rows, D, 900 + D)
    yl = ak.ak_layernorm_fwd(xl.to(dev), g.to(dev), b.to(dev))
    refl = oracle.layernorm(synth.to_bits(xl), synth.to_bits(g), synth.to_bits(b), 1e-5)
    assert (np.abs(widen(yl) - refl) / np.maximum(1.0, np.abs(refl))).max() <= 1.6e-2
print("no clusters ok")
"""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, AK_DISABLE_CLUSTERS="1")
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=900)
    assert r.returncode == 0 and "no clusters ok" in r.stdout, r.stdout[-2000:] + r.stderr[-4000:]

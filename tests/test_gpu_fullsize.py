"""Full-size benchmark shapes in the launch configuration the benchmark times.  Tensors of up to
1 GiB (every shape of the benchmark configurations but two) are compared with the fp64 CPU
checker element by element over ALL rows, in row chunks; the two larger ones (262144 x 4096,
16384 x 128256) over 1024 sampled rows plus first / middle / last.  Every shape is also checked
through properties that hold at any size (finite, row sums, mean = fp64 mean of the per-row
losses) and for bitwise run-to-run determinism.  Inputs are generated on the device from a
seed; their bit patterns are copied back chunk by chunk so both sides see identical bits."""
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import synth
from parity import assert_bf16_close, assert_close_on_device, assert_loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"
ALL_ROWS_UP_TO = 1 << 29      # elements: tensors of up to 1 GiB (bf16) are compared whole
CHUNK_ELEMS = 1 << 25         # elements per chunk handed to the checker (256 MB of fp64)


def _row_chunks(rows, D, sample=1024, seed=0):
    """Index tensors (on the device) of the rows to compare, chunk by chunk: every row when the
    tensor has at most ALL_ROWS_UP_TO elements, else `sample` random rows plus first, middle, last."""
    if rows * D <= ALL_ROWS_UP_TO:
        idx = np.arange(rows, dtype=np.int64)
    else:
        idx = _sample_rows(rows, n=sample, seed=seed)
    per = max(1, CHUNK_ELEMS // D)
    return [torch.from_numpy(idx[i:i + per]).to(DEV) for i in range(0, len(idx), per)]


def _sample_rows(rows, n=40, seed=0):
    rng = np.random.default_rng(seed)
    idx = {0, rows - 1, rows // 2}
    idx.update(int(i) for i in rng.integers(0, rows, size=min(n, rows)))
    return np.array(sorted(idx), dtype=np.int64)


def _free():
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


@pytest.mark.parametrize("rows,D", [(8192, 1024), (8192, 2048), (8192, 4096), (8192, 8192),
                                    (8192, 16384), (65536, 4096), (262144, 4096), (8192, 4099),
                                    (4096, 65536), (2048, 128256), (16, 128256), (512, 262144)])
def test_rmsnorm_full_size(rows, D):
    x, w = synth.rmsnorm_inputs(rows, D, synth.case_seed(2, D + rows), device=DEV)
    y = ak.ak_rmsnorm_fwd(x, w, eps=1e-6)
    y2 = ak.ak_rmsnorm_fwd(x, w, eps=1e-6)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    del y2
    for it in _row_chunks(rows, D, seed=D):
        ref = oracle.rmsnorm(synth.to_bits(x[it]), synth.to_bits(w), 1e-6)
        assert_close_on_device(y[it], ref, f"rmsnorm {rows}x{D} rows {int(it[0])}..{int(it[-1])}")
    # property: mean square of y / w is 1 (eps is negligible for N(0,1) rows)
    for r0 in range(0, rows, 32768):
        blk = y[r0:r0 + 32768].float() / w.float()[None, :]
        ms = (blk * blk).mean(dim=-1)
        assert torch.isfinite(blk).all()
        assert bool(((ms - 1).abs() < 2e-2).all())
    del x, y
    _free()


@pytest.mark.parametrize("rows,D", [(16384, 512), (16384, 1024), (16384, 2048), (16384, 4096),
                                    (16384, 8192), (16384, 32768), (262144, 4096), (4096, 4099),
                                    (4096, 65536), (4096, 128256), (16, 128256), (1, 128256), (512, 262144),
                                    (4096, 128257), (16, 50257)])
def test_softmax_full_size(rows, D):
    x = synth.softmax_inputs(rows, D, synth.case_seed(3, D + rows), device=DEV)
    y = ak.ak_softmax_fwd(x)
    y2 = ak.ak_softmax_fwd(x)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    del y2
    chunks = _row_chunks(rows, D, seed=D)
    if rows * D > ALL_ROWS_UP_TO:   # make sure masked rows are among the samples
        chunks.append(torch.nonzero(x[:, -1].float() == float("-inf")).flatten()[:8])
    for it in chunks:
        if it.numel():
            ref = oracle.softmax(synth.to_bits(x[it]))
            assert_close_on_device(y[it], ref, f"softmax {rows}x{D} rows {int(it[0])}..{int(it[-1])}")
    for r0 in range(0, rows, 16384):
        blk = y[r0:r0 + 16384].float()
        assert torch.isfinite(blk).all() and bool((blk >= 0).all())
        assert bool(((blk.sum(dim=-1) - 1).abs() < 6e-3).all())
        assert bool((blk[x[r0:r0 + 16384].float() == float("-inf")] == 0).all())
    del x, y
    _free()


@pytest.mark.parametrize("rows,V", [(4096, 32000), (4096, 50304), (4096, 128256),
                                    (16384, 128256), (4096, 128257), (16, 128256)])
def test_xent_full_size(rows, V):
    logits, targets = synth.xent_inputs(rows, V, synth.case_seed(4, V + rows), device=DEV)
    loss, mean = ak.ak_xent_fwd(logits, targets)
    loss2, mean2 = ak.ak_xent_fwd(logits, targets)
    torch.cuda.synchronize()
    assert torch.equal(loss.view(torch.int32), loss2.view(torch.int32))
    assert torch.equal(mean.view(torch.int32), mean2.view(torch.int32))
    ref_all, idx_all = [], []
    for it in _row_chunks(rows, V, seed=V):
        ref_rows, _, _ = oracle.xent(synth.to_bits(logits[it]), targets[it].cpu().numpy())
        assert_loss_close(loss[it], ref_rows, f"xent {rows}x{V} rows {int(it[0])}..{int(it[-1])}")
        ref_all.append(ref_rows)
        idx_all.append(it)
    valid = targets != -100
    if rows * V <= ALL_ROWS_UP_TO:   # every row was checked: the checker's own mean is at hand
        ref_rows = np.concatenate(ref_all)
        ref_mean = ref_rows[valid.cpu().numpy()].sum() / int(valid.sum())
        assert_loss_close(mean, np.array([ref_mean]), f"xent {rows}x{V} mean against the checker")
    assert bool((loss[~valid] == 0).all()) and bool((loss[valid] > 0).all())
    want_mean = loss[valid].double().sum().item() / int(valid.sum())
    assert abs(mean.item() - want_mean) <= 1e-6 * want_mean
    if rows >= 4096:
        assert abs(mean.item() - (math.log(V) + 2.0)) < 0.2   # E[loss] for N(0, 2^2) logits
    del logits
    _free()


@pytest.mark.parametrize("rows,D", [(8192, 4096), (4096, 5120), (8192, 8192), (65536, 4096), (4096, 32768),
                                    (8192, 4099), (4096, 65536), (2048, 128256), (16, 128256), (512, 262144)])
def test_layernorm_full_size(rows, D):
    x, g, b = synth.layernorm_inputs(rows, D, synth.case_seed(6, D + rows), device=DEV)
    y = ak.ak_layernorm_fwd(x, g, b, eps=1e-5)
    y2 = ak.ak_layernorm_fwd(x, g, b, eps=1e-5)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))
    del y2
    for it in _row_chunks(rows, D, seed=D):
        ref = oracle.layernorm(synth.to_bits(x[it]), synth.to_bits(g), synth.to_bits(b), 1e-5)
        assert_close_on_device(y[it], ref, f"layernorm {rows}x{D} rows {int(it[0])}..{int(it[-1])}", tight=False)
    # property: (y - beta) / gamma has zero mean and unit variance in every row
    for r0 in range(0, rows, 16384):
        z = (y[r0:r0 + 16384].float() - b.float()[None, :]) / g.float()[None, :]
        assert torch.isfinite(z).all()
        assert bool((z.mean(dim=-1).abs() < 2e-2).all())
        assert bool((((z * z).mean(dim=-1)) - 1).abs().max() < 3e-2)
    del x, y
    _free()


@pytest.mark.parametrize("rows,D", [(16384, 4096), (8192, 8192), (65536, 1024), (65536, 8192), (4096, 128256),
                                    (8192, 4099)])
def test_rowsum_full_size(rows, D):
    x, _, _ = synth.layernorm_inputs(rows, D, synth.case_seed(8, D + rows), device=DEV)
    s = ak.ak_rowsum_fwd(x)
    s2 = ak.ak_rowsum_fwd(x)
    torch.cuda.synchronize()
    assert torch.equal(s.view(torch.int32), s2.view(torch.int32))
    for it in _row_chunks(rows, D, seed=D):
        xb = synth.to_bits(x[it])
        ref = oracle.rowsum(xb)
        mag = x[it].double().abs().sum(dim=-1).cpu().numpy()
        err = np.abs(s[it].cpu().double().numpy() - ref)
        assert float(np.max(err / (1e-6 * mag + 2.0 ** -24 * np.abs(ref)))) <= 1.0
    # property at any size: agrees with a float64 sum done by another library on the device
    for r0 in range(0, rows, 8192):
        want = x[r0:r0 + 8192].double().sum(dim=-1)
        absx = x[r0:r0 + 8192].double().abs().sum(dim=-1)
        assert bool(((s[r0:r0 + 8192].double() - want).abs() <= 1e-6 * absx + 1e-6 * want.abs()).all())
    del x
    _free()


@pytest.mark.parametrize("dtype,S", [(torch.float16, 2048), (torch.float16, 4096), (torch.bfloat16, 4096),
                                     (torch.float32, 4096)])
def test_rope_full_size(dtype, S):
    n_seq, Dh = 64, 128                                    # 2 x 32 heads, the benchmark's layout
    x = synth.rope_inputs(n_seq, S, Dh, synth.case_seed(18, S), device=DEV, dtype=dtype)
    y = ak.ak_rope_fwd(x)
    y2 = ak.ak_rope_fwd(x)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.uint8), y2.view(torch.uint8))
    del y2
    name = synth.DTYPE_NAMES[dtype]
    tol = {torch.bfloat16: 1.6e-2, torch.float16: 1e-3, torch.float32: 1e-5}[dtype]
    for p in (0, 1, S // 2, S - 1, 777):                   # sampled positions, every sequence
        ref = oracle.rope(synth.to_elems(x[:, p:p + 1].contiguous()), name, pos_offset=p)
        got = y[:, p:p + 1].cpu().double().numpy()
        assert float(np.max(np.abs(got - ref) / (tol * np.maximum(1.0, np.abs(ref))))) <= 1.0
    # property at any size: a rotation keeps the length of every pair
    xf, yf = x.float(), y.float()
    n_in = xf[..., 0::2] ** 2 + xf[..., 1::2] ** 2
    n_out = yf[..., 0::2] ** 2 + yf[..., 1::2] ** 2
    rel = {torch.bfloat16: 2e-2, torch.float16: 3e-3, torch.float32: 1e-5}[dtype]
    assert bool(((n_out - n_in).abs() <= rel * n_in + 1e-6).all())
    del x, y
    _free()


@pytest.mark.parametrize("dtype", [torch.float16, torch.float32])
def test_dtype_variants_full_size(dtype):
    name = synth.DTYPE_NAMES[dtype]
    from parity import assert_close_dt
    x, w = synth.rmsnorm_inputs(8192, 8192, synth.case_seed(12, 1), device=DEV, dtype=dtype)
    y = ak.ak_rmsnorm_fwd_dt(x, w)
    it = torch.from_numpy(_sample_rows(8192, seed=1)).to(DEV)
    assert_close_dt(y[it], oracle.rmsnorm_dt(synth.to_elems(x[it]), synth.to_elems(w), 1e-6, name), f"rmsnorm {name} full")
    del x, y
    _free()
    xs = synth.softmax_inputs(16384, 8192, synth.case_seed(13, 1), device=DEV, dtype=dtype)
    y = ak.ak_softmax_fwd_dt(xs)
    it = torch.from_numpy(_sample_rows(16384, seed=2)).to(DEV)
    assert_close_dt(y[it], oracle.softmax_dt(synth.to_elems(xs[it]), name), f"softmax {name} full")
    assert bool(((y.float().sum(dim=-1) - 1).abs() < 2e-3).all())
    del xs, y
    _free()
    V = 128256 if dtype == torch.float16 else 50304
    lg, tg = synth.xent_inputs(4096, V, synth.case_seed(14, 1), device=DEV, dtype=dtype)
    loss, mean = ak.ak_xent_fwd_dt(lg, tg)
    idx = _sample_rows(4096, seed=3)
    it = torch.from_numpy(idx).to(DEV)
    ref_rows, _, _ = oracle.xent_dt(synth.to_elems(lg[it]), tg[it].cpu().numpy(), name)
    assert_loss_close(loss[it], ref_rows, f"xent {name} full")
    valid = tg != -100
    want_mean = loss[valid].double().sum().item() / int(valid.sum())
    assert abs(mean.item() - want_mean) <= 1e-6 * want_mean
    del lg
    _free()


def test_vocab_parallel_full_size_eight_ranks():
    from paper_2603_21331_b200 import parallel
    rows, V, world = 4096, 128256, 8
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(16, 1), device=DEV)
    parts = []
    for rank in range(world):
        b, e = parallel.shard_vocab(V, rank, world)
        parts.append(ak.ak_xent_vp_partial(lg[:, b:e].contiguous(), tg, b, V, 1))
    loss, mean = ak.ak_xent_vp_merge(torch.stack(parts).contiguous(), tg, V)
    idx = _sample_rows(rows, seed=4)
    it = torch.from_numpy(idx).to(DEV)
    ref_rows, _, _ = oracle.xent(synth.to_bits(lg[it]), tg[it].cpu().numpy())
    assert_loss_close(loss[it], ref_rows, "vocabulary-parallel xent, 8 shards, sampled rows")
    # and against the single-GPU kernel on the unsharded logits: same loss up to the merge's rounding
    single, smean = ak.ak_xent_fwd(lg, tg)
    assert bool(((loss - single).abs() <= 2e-6 * single.abs().clamp(min=1.0)).all())
    assert abs(mean.item() - smean.item()) <= 2e-6 * abs(smean.item())
    del lg
    _free()

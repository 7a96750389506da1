"""Vocabulary-parallel cross-entropy on one GPU: the ranks' shards are processed one after the
other (no kernel waits on another), their partial buffers stacked as the all-gather would, and
the merge compared with the fp64 CPU checker on the FULL logits."""
import os

import numpy as np
import pytest
import torch

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import parallel, synth
from parity import assert_loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"
NAME = synth.DTYPE_NAMES


def _vp(logits_dev, targets_dev, world, nsplit):
    rows, V = logits_dev.shape
    if nsplit == 0:
        nsplit = ak.ak_xent_vp_nsplit(rows, parallel.shard_vocab(V, 0, world)[1])
    parts = []
    for rank in range(world):
        b, e = parallel.shard_vocab(V, rank, world)
        shard = logits_dev[:, b:e].contiguous()
        parts.append(ak.ak_xent_vp_partial(shard, targets_dev, b, V, nsplit))
    return ak.ak_xent_vp_merge(torch.stack(parts).contiguous(), targets_dev, V)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float16, torch.float32])
@pytest.mark.parametrize("rows,V,world", [(64, 1000, 2), (33, 4099, 3), (24, 32000, 8), (8, 128256, 8),
                                          (6, 128257, 4), (7, 9, 2), (300, 2048, 1), (1500, 4096, 2)])
def test_vocab_parallel_matches_checker_and_single_gpu(rows, V, world, dtype):
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(16, rows * 131 + V), dtype=dtype, ignore_frac=0.1)
    ref_rows, ref_mean, n = oracle.xent_dt(synth.to_elems(lg), tg.numpy(), NAME[dtype])
    ld, td = lg.to(DEV), tg.to(DEV)
    for nsplit in (0, 1, 3):
        loss, mean = _vp(ld, td, world, nsplit)
        torch.cuda.synchronize()
        assert_loss_close(loss, ref_rows, f"vp xent {NAME[dtype]} {rows}x{V} world {world} nsplit {nsplit}")
        assert bool((loss[td == -100] == 0).all())
        if n > 0:
            assert_loss_close(mean, np.array([ref_mean]), "vp xent mean")
    # one rank, one slice is the single-GPU row kernel's arithmetic: same bits
    one, one_mean = _vp(ld, td, 1, 1)
    row, row_mean = ak.ak_xent_fwd_dt(ld, td, path=ak.AK_XENT_ROW)
    assert torch.equal(one.view(torch.int32), row.view(torch.int32))
    assert torch.equal(one_mean.view(torch.int32), row_mean.view(torch.int32))


def test_vocab_parallel_conventions():
    rows, V, world = 12, 1000, 4
    lg, tg = synth.xent_inputs(rows, V, 1717)
    tg[0] = -100
    tg[1] = V          # out of range: NaN, counted
    tg[2] = -5
    tg[3] = 0          # first column of rank 0
    tg[4] = V - 1      # last column of the last rank
    tg[5] = parallel.shard_vocab(V, 1, world)[0]   # first column of rank 1
    ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(lg), tg.numpy())
    loss, mean = _vp(lg.to(DEV), tg.to(DEV), world, 2)
    assert_loss_close(loss, ref_rows, "vp conventions")
    assert np.isnan(ref_mean) and bool(torch.isnan(mean).all())
    # all rows ignored: mean NaN, losses 0
    tg[:] = -100
    loss, mean = _vp(lg.to(DEV), tg.to(DEV), world, 1)
    assert bool((loss == 0).all()) and bool(torch.isnan(mean).all())
    # a target column owned by no shard (the caller passed wrong shard bounds) surfaces as NaN
    lg2, tg2 = synth.xent_inputs(4, 64, 1718, ignore_frac=0.0)
    tg2[:] = 40
    part = ak.ak_xent_vp_partial(lg2[:, :32].contiguous().to(DEV), tg2.to(DEV), 0, 64, 1)
    loss, _ = ak.ak_xent_vp_merge(part[None].contiguous(), tg2.to(DEV), 64)
    assert bool(torch.isnan(loss).all())


def test_vocab_parallel_adversarial_and_determinism():
    rows, V, world = 20, 4096, 4
    for kind in synth.ADVERSARIAL_KINDS:
        x, hot = synth.adversarial_rows(kind, rows, V, synth.case_seed(17, V))
        t = hot.clone()
        t[1::2] = (t[1::2] + 1) % V
        ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(x), t.numpy())
        loss, mean = _vp(x.to(DEV), t.to(DEV), world, 2)
        assert torch.isfinite(loss).all() and bool((loss >= 0).all())
        assert_loss_close(loss, ref_rows, f"vp adversarial {kind}")
        assert_loss_close(mean, np.array([ref_mean]), f"vp adversarial mean {kind}")
        again, mean2 = _vp(x.to(DEV), t.to(DEV), world, 2)
        assert torch.equal(loss.view(torch.int32), again.view(torch.int32))
        assert torch.equal(mean.view(torch.int32), mean2.view(torch.int32))


@pytest.mark.parametrize("rows,world,ignore", [(1, 2, 0.0), (127, 8, 0.1), (1024, 8, 0.1), (1025, 3, 0.3), (4096, 8, 0.05),
                                               (8192, 2, 0.0), (300, 8, 1.0)])
def test_vocab_parallel_merge_and_mean_in_one_launch(rows, world, ignore):
    """Up to 8192 rows the merge and the fixed-order mean run as one cluster launch.  Its losses
    are, bit for bit, those of the merge kernel alone (what `want_mean=False` runs), and its mean
    is, bit for bit, the fixed-order mean of those losses (the row-shard kernels: fp64 sum and count
    of the counted rows, then their quotient); larger batches take two kernels and agree too."""
    if os.environ.get("AK_DISABLE_CLUSTERS", "0") not in ("", "0"):
        pytest.skip("the cluster layouts are switched off in this environment")
    V = 2048 * world
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(41, rows * 7 + world), ignore_frac=min(ignore, 0.999))
    if ignore >= 1.0:
        tg[:] = -100
    ld, td = lg.to(DEV), tg.to(DEV)
    parts = []
    for rank in range(world):
        b, e = parallel.shard_vocab(V, rank, world)
        parts.append(ak.ak_xent_vp_partial(ld[:, b:e].contiguous(), td, b, V, 1))
    stack = torch.stack(parts).contiguous()
    n0 = ak.ak_launch_count()
    loss, mean = ak.ak_xent_vp_merge(stack, td, V)
    torch.cuda.synchronize()
    assert ak.ak_launch_count() - n0 == 1
    loss_only, none = ak.ak_xent_vp_merge(stack, td, V, want_mean=False)
    assert none is None
    assert torch.equal(loss.view(torch.int32), loss_only.view(torch.int32))
    want = ak.ak_xent_mean_merge(ak.ak_xent_sum_count(loss_only, td).view(1, 2))
    torch.cuda.synchronize()
    assert torch.equal(mean.view(torch.int32), want.view(torch.int32)) or (torch.isnan(mean).all() and torch.isnan(want).all())
    ref_rows, ref_mean, n = oracle.xent(synth.to_bits(lg), tg.numpy())
    assert_loss_close(loss, ref_rows, f"vp merge+mean {rows} rows world {world}")
    if n > 0:
        assert abs(float(mean) - ref_mean) <= 1e-5 * max(1.0, abs(ref_mean))
    else:
        assert torch.isnan(mean).all()
    assert ak.ak_wait_timeouts() == 0

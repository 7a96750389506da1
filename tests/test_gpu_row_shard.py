"""The row-shard mean on one GPU: the batch is cut into row blocks with ``parallel.shard_rows``,
each emulated rank runs the cross-entropy kernel and ``ak_xent_sum_count`` on its block (one
after the other; no kernel waits on another), the 16-byte pairs are stacked in rank order as the
all-gather would deliver them, and ``ak_xent_mean_merge`` gives the mean, compared with the fp64
CPU checker on the whole batch.  A one-rank NCCL group then runs ``parallel.global_xent_mean``
and ``parallel.vocab_parallel_xent`` themselves, on a stream that is not the current one."""
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

import oracle
import paper_2603_21331_b200 as ak
from paper_2603_21331_b200 import parallel, synth
from parity import assert_loss_close

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _sharded_mean(ld, td, world, ignore_index=-100):
    rows = ld.shape[0]
    pairs, losses = [], []
    for rank in range(world):
        b, e = parallel.shard_rows(rows, rank, world)
        if e > b:
            loss, _ = ak.ak_xent_fwd(ld[b:e], td[b:e], ignore_index, want_mean=False)
        else:
            loss = torch.empty((0,), dtype=torch.float32, device=ld.device)
        losses.append(loss)
        pairs.append(ak.ak_xent_sum_count(loss, td[b:e], ignore_index))
    stacked = torch.stack(pairs).contiguous()
    return ak.ak_xent_mean_merge(stacked), stacked, torch.cat(losses)


@pytest.mark.parametrize("rows,V", [(37, 1000), (600, 4099), (3000, 512), (5, 32000)])
@pytest.mark.parametrize("world", [1, 2, 3, 8])
def test_row_shard_mean_matches_full_batch(rows, V, world):
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(17, rows + V), ignore_frac=0.2)
    ref_rows, ref_mean, n = oracle.xent(synth.to_bits(lg), tg.numpy())
    ld, td = lg.to(DEV), tg.to(DEV)
    mean, pairs, loss = _sharded_mean(ld, td, world)
    torch.cuda.synchronize()
    assert_loss_close(loss, ref_rows, f"row-shard losses {rows}x{V} world {world}")
    assert_loss_close(mean, np.array([ref_mean]), f"row-shard mean {rows}x{V} world {world}")
    assert pairs[:, 1].sum().item() == n                     # counts are exact integers
    # the pair of a block is the fp64 sum of ITS fp32 losses; the merge adds the pairs in rank order
    got = loss.cpu().double().numpy()
    keep = tg.numpy() != -100
    total = 0.0
    for rank in range(world):
        b, e = parallel.shard_rows(rows, rank, world)
        blk = float(np.sum(got[b:e][keep[b:e]], dtype=np.float64))
        assert abs(pairs[rank, 0].item() - blk) <= 1e-12 * max(1.0, abs(blk))
        total += pairs[rank, 0].item()
    assert mean.item() == np.float32(total / n)
    # same bits on a second and third run
    for _ in range(2):
        again, pairs2, _ = _sharded_mean(ld, td, world)
        assert torch.equal(again.view(torch.int32), mean.view(torch.int32))
        assert torch.equal(pairs2.view(torch.int64), pairs.view(torch.int64))


def test_row_shard_mean_degenerate_blocks():
    rows, V, world = 10, 257, 4
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(17, 99), ignore_frac=0.0)
    tg[0:3] = -100                      # rank 0's block (rows 0..2) counts nothing
    ld, td = lg.to(DEV), tg.to(DEV)
    ref_rows, ref_mean, n = oracle.xent(synth.to_bits(lg), tg.numpy())
    mean, pairs, _ = _sharded_mean(ld, td, world)
    assert pairs[0, 0].item() == 0.0 and pairs[0, 1].item() == 0.0
    assert_loss_close(mean, np.array([ref_mean]), "mean with an all-ignored block")
    # more ranks than rows: empty blocks contribute (0, 0)
    mean16, pairs16, _ = _sharded_mean(ld, td, 16)
    assert pairs16.shape == (16, 2) and bool((pairs16[10:] == 0).all())
    assert_loss_close(mean16, np.array([ref_mean]), "mean with empty blocks")
    # every block ignored: 0 / 0 = NaN, as for the single-GPU mean
    t_all = torch.full_like(td, -100)
    m, p, _ = _sharded_mean(ld, t_all, 3)
    assert bool((p == 0).all()) and torch.isnan(m).all()
    # a target out of range makes its row's loss NaN and counts: the mean is NaN on every rank
    t_bad = td.clone()
    t_bad[7] = V + 5
    m, p, _ = _sharded_mean(ld, t_bad, 4)
    assert torch.isnan(m).all() and torch.isnan(p[:, 0]).sum().item() == 1
    assert p[:, 1].sum().item() == rows - 3
    # an empty list of pairs
    assert torch.isnan(ak.ak_xent_mean_merge(torch.empty((0, 2), dtype=torch.float64, device=DEV))).all()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_one_rank_nccl_group_on_a_side_stream():
    """``global_xent_mean`` and ``vocab_parallel_xent`` through a real (one-rank) NCCL group, with
    their work on a stream other than the current one: producer kernel, collective and consumer
    kernel must be ordered on THAT stream."""
    rows, V = 700, 4096
    lg, tg = synth.xent_inputs(rows, V, synth.case_seed(17, 7), ignore_frac=0.1)
    ref_rows, ref_mean, _ = oracle.xent(synth.to_bits(lg), tg.numpy())
    ld, td = lg.to(DEV), tg.to(DEV)
    started = not dist.is_initialized()
    if started:
        dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{_free_port()}", rank=0, world_size=1,
                                device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        side = torch.cuda.Stream()
        loss, _ = ak.ak_xent_fwd(ld, td, want_mean=False)
        side.wait_stream(torch.cuda.current_stream())
        for _ in range(3):
            # a long kernel on the side stream ahead of the sequence: anything that ordered itself
            # against the current stream instead would run too early
            filler = torch.empty((64 << 20,), dtype=torch.float32, device=DEV)
            with torch.cuda.stream(side):
                filler.fill_(1.0)
                scratch_loss = loss.clone()
            mean = parallel.global_xent_mean(scratch_loss, td, stream=side)
            rows_vp, mean_vp = parallel.vocab_parallel_xent(ld, td, 0, V, stream=side.cuda_stream)
            side.synchronize()
            assert_loss_close(mean, np.array([ref_mean]), "global_xent_mean on a side stream")
            assert_loss_close(rows_vp, ref_rows, "vocab_parallel_xent rows on a side stream")
            assert_loss_close(mean_vp, np.array([ref_mean]), "vocab_parallel_xent mean on a side stream")
            del filler
    finally:
        if started:
            dist.destroy_process_group()

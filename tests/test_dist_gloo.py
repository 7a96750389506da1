"""World-size-2 CPU test (gloo) of the row-shard host logic: block sharding, the 16-byte
(sum, count) exchange in rank order, and the rank-order merge, against the full-batch
mean of the CPU checker.  No GPU is involved; per-rank losses come from the checker."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import oracle
from paper_2603_21331_b200 import parallel, synth


def merge_pairs_host(pairs: torch.Tensor) -> float:
    """Rank-order merge of gathered (sum, count) pairs on the host: what the library's merge
    kernel computes, written out here so the exchange can be checked without a GPU."""
    total, count = 0.0, 0.0
    for s, c in pairs.double().cpu().tolist():
        total += s
        count += c
    return total / count if count > 0 else float("nan")


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, rows, V, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        logits, targets = synth.xent_inputs(rows, V, seed=4242, ignore_frac=0.25)
        b, e = parallel.shard_rows(rows, rank, world)
        loss, _, n = oracle.xent(synth.to_bits(logits[b:e]), targets[b:e].numpy())
        keep = targets[b:e].numpy() != -100
        pair = torch.tensor([float(np.sum(loss[keep])), float(n)], dtype=torch.float64)
        pairs = parallel.gather_pairs(pair)
        assert pairs.shape == (world, 2)
        assert pairs[rank, 0].item() == pair[0].item() and pairs[rank, 1].item() == pair[1].item()
        mean = merge_pairs_host(pairs)
        np.save(os.path.join(out_dir, f"mean{rank}.npy"), np.array([mean]))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("rows", [37, 2])
def test_row_sharded_mean_two_ranks(tmp_path, rows):
    V, world = 257, 2
    mp.spawn(_worker, args=(world, _free_port(), rows, V, str(tmp_path)), nprocs=world, join=True)
    means = [np.load(tmp_path / f"mean{r}.npy")[0] for r in range(world)]
    assert means[0] == means[1]                        # bit-identical on every rank
    logits, targets = synth.xent_inputs(rows, V, seed=4242, ignore_frac=0.25)
    _, full_mean, _ = oracle.xent(synth.to_bits(logits), targets.numpy())
    assert means[0] == pytest.approx(full_mean, rel=1e-14, nan_ok=True)


def test_shard_rows_covers_everything_once():
    for rows in (0, 1, 7, 8, 4096, 4099):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_rows(rows, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == rows
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            sizes = [e - b for b, e in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        parallel.shard_rows(4, 2, 2)


def test_merge_pairs_host_conventions():
    assert np.isnan(merge_pairs_host(torch.zeros((2, 2), dtype=torch.float64)))
    p = torch.tensor([[3.0, 2.0], [0.0, 0.0], [9.0, 2.0]], dtype=torch.float64)
    assert merge_pairs_host(p) == 3.0


def _vp_worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        rows, nsplit = 5, 3
        # a recognisable partial buffer: value encodes (rank, row, slot, component)
        part = torch.arange(rows * (nsplit + 1) * 2, dtype=torch.float32).view(rows, nsplit + 1, 2) + 1000.0 * rank
        parts = parallel.gather_partials(part)
        assert parts.shape == (world, rows, nsplit + 1, 2)
        for k in range(world):
            assert torch.equal(parts[k], part - 1000.0 * rank + 1000.0 * k)   # rank order, layout kept
        np.save(os.path.join(out_dir, f"parts{rank}.npy"), parts.numpy())
    finally:
        dist.destroy_process_group()


def test_vocab_parallel_exchange_two_ranks(tmp_path):
    """The one exchange of the vocabulary-parallel cross-entropy: every rank ends with all
    ranks' partial buffers, in rank order, bit-identical everywhere."""
    world = 2
    mp.spawn(_vp_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    a, b = (np.load(tmp_path / f"parts{r}.npy") for r in range(world))
    assert np.array_equal(a, b)


def test_shard_vocab_tiles_the_vocabulary_with_aligned_starts():
    for V in (1, 9, 1000, 4099, 32000, 128256, 128257):
        for world in (1, 2, 3, 8):
            spans = [parallel.shard_vocab(V, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == V
            assert all(spans[i][1] == spans[i + 1][0] for i in range(world - 1))
            assert all(b % 8 == 0 or b == V for b, _ in spans)
    with pytest.raises(ValueError):
        parallel.shard_vocab(8, 3, 2)

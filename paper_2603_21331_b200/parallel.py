"""Row-sharded execution across GPUs (one process per GPU, ``torch.distributed``).

Rows are independent, so RMSNorm, softmax and the per-row cross-entropy losses need no
communication at all when each rank holds a block of rows.  Only the scalar
cross-entropy mean has an exchange step: each rank contributes the 16-byte pair
(fp64 sum of its counted losses, count); the pairs are all-gathered and added in rank
order by the library's merge kernel, so every rank obtains the same bits regardless of
the collective's internal algorithm.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def shard_rows(rows: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block [begin, end) of ``rows`` owned by ``rank``; sizes differ by at most 1."""
    if world < 1 or not (0 <= rank < world) or rows < 0:
        raise ValueError("bad shard request")
    base, extra = divmod(rows, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def gather_pairs(local_pair: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather the per-rank (sum, count) pairs -> [world, 2] float64, in rank order."""
    if local_pair.dtype != torch.float64 or local_pair.numel() != 2:
        raise TypeError("local_pair must be a float64 tensor with 2 elements")
    world = dist.get_world_size(group)
    out = torch.empty((world, 2), dtype=torch.float64, device=local_pair.device)
    dist.all_gather_into_tensor(out.view(-1), local_pair.view(-1).contiguous(), group=group)
    return out


def shard_vocab(V: int, rank: int, world: int) -> Tuple[int, int]:
    """Contiguous block [begin, end) of the vocabulary owned by ``rank``.  Block starts are
    multiples of 8 columns (16-byte aligned shards for the 16-bit types); the last rank takes
    the remainder."""
    if world < 1 or not (0 <= rank < world) or V < 0:
        raise ValueError("bad shard request")
    per = -(-V // world)
    per = -(-per // 8) * 8
    begin = min(V, rank * per)
    return begin, min(V, begin + per)


def gather_partials(partial: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather the per-rank partial buffers [rows, nsplit + 1, 2] -> [world, rows, nsplit + 1, 2]
    in rank order (the only exchange of the vocabulary-parallel cross-entropy)."""
    if partial.dtype != torch.float32 or partial.dim() != 3 or partial.shape[2] != 2:
        raise TypeError("partial must be a float32 tensor [rows, nsplit + 1, 2]")
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(partial.shape), dtype=torch.float32, device=partial.device)
    dist.all_gather_into_tensor(out.view(-1), partial.contiguous().view(-1), group=group)
    return out


def _stream_of(stream, device: torch.device) -> "torch.cuda.Stream":
    """``stream`` (None = the current one, a torch stream, or a raw cudaStream_t handle) as a torch
    stream object of ``device``."""
    if stream is None:
        return torch.cuda.current_stream(device)
    if isinstance(stream, torch.cuda.Stream):
        return stream
    return torch.cuda.ExternalStream(int(stream), device=device)


def vocab_parallel_xent(logits_shard: torch.Tensor, targets: torch.Tensor, vocab_start: int, V_total: int,
                        ignore_index: int = -100, group=None, stream=None, nsplit: int = 0):
    """Cross-entropy of [rows, V_total] logits whose columns are sharded over the ranks of
    ``group``: this rank passes its [rows, V_local] block and its first column.  Returns
    (loss_rows, loss_mean), bit-identical on every rank.  ``nsplit`` must agree across ranks;
    0 derives it from (rows, largest shard), which is the same everywhere for block shards."""
    from . import binding
    rows, V_local = logits_shard.shape
    if nsplit == 0:
        world = dist.get_world_size(group)
        nsplit = binding.ak_xent_vp_nsplit(rows, shard_vocab(V_total, 0, world)[1])
    # The collective orders itself against the CURRENT stream, so `stream` is made current for
    # the whole sequence: partial kernel -> all-gather -> merge kernel run in that order on it.
    st = _stream_of(stream, logits_shard.device)
    with torch.cuda.stream(st):
        part = binding.ak_xent_vp_partial(logits_shard, targets, vocab_start, V_total, nsplit, ignore_index,
                                          stream=st)
        parts = gather_partials(part, group)
        return binding.ak_xent_vp_merge(parts, targets, V_total, ignore_index, stream=st)


def global_xent_mean(loss_rows: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                     group=None, stream=None) -> torch.Tensor:
    """Mean cross-entropy over all ranks' rows (device tensors; kernels from libak).  The two
    kernels and the 16-byte all-gather between them run on ``stream`` (default: the current one),
    which is made current for the sequence because the collective orders itself against the
    current stream."""
    from . import binding
    st = _stream_of(stream, loss_rows.device)
    with torch.cuda.stream(st):
        pair = binding.ak_xent_sum_count(loss_rows, targets, ignore_index, stream=st)
        pairs = gather_pairs(pair, group)
        return binding.ak_xent_mean_merge(pairs, stream=st)

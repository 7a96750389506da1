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


def merge_pairs_host(pairs: torch.Tensor) -> float:
    """Rank-order merge of gathered pairs on the host (CPU tensors): the same arithmetic,
    in the same order, as the library's merge kernel.  Used where no GPU is involved."""
    total, count = 0.0, 0.0
    for s, c in pairs.double().cpu().tolist():
        total += s
        count += c
    return total / count if count > 0 else float("nan")


def global_xent_mean(loss_rows: torch.Tensor, targets: torch.Tensor, ignore_index: int = -100,
                     group=None, stream=None) -> torch.Tensor:
    """Mean cross-entropy over all ranks' rows (device tensors; kernels from libak)."""
    from . import binding
    lib = binding.lib()
    st = binding._stream_ptr(stream)
    pair = torch.empty((2,), dtype=torch.float64, device=loss_rows.device)
    binding._check(lib.ak_xent_sum_count(loss_rows.data_ptr(), targets.data_ptr(), ignore_index,
                                         loss_rows.numel(), pair.data_ptr(), st), "ak_xent_sum_count")
    pairs = gather_pairs(pair, group)
    mean = torch.empty((1,), dtype=torch.float32, device=loss_rows.device)
    binding._check(lib.ak_xent_mean_merge(pairs.data_ptr(), pairs.shape[0], mean.data_ptr(), st),
                   "ak_xent_mean_merge")
    return mean

"""Element-range sharding of the averaging step over several GPUs (one process per GPU).

Every rank holds the same index range [j0, j1) of all M replicas.  Sums of squares add over
disjoint ranges, so one all-gather of a [K, M] table of doubles is the only exchange:

    local sums (grawa_layer_sumsq)  ->  all-gather  ->  grawa_step_from_layer_sums on the local range

The tables are added in rank order inside the library's kernel, so every rank computes the same
weights bit for bit; centre and pull are local.  torch.distributed carries the all-gather (NCCL on
GPUs); everything else runs in the library's kernels.
"""
from __future__ import annotations

import numpy as np

from . import binding


def shard_range(n: int, world: int, rank: int, align: int = 4):
    """Element range [j0, j1) of `rank`: an even split of the `align`-element blocks of [0, n)."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    blocks = (n + align - 1) // align
    b0 = blocks * rank // world
    b1 = blocks * (rank + 1) // world
    return min(n, b0 * align), min(n, b1 * align)


def local_layer_table(layer_offsets, j0: int, j1: int) -> np.ndarray:
    """Layer table of the range [j0, j1): the global offsets clipped to the range and shifted to it.
    Layers without elements in the range become empty layers (same number of layers on every rank)."""
    off = np.asarray(layer_offsets, dtype=np.int64)
    return np.clip(off, j0, j1) - j0


def exchange_layer_sums(local, group=None):
    """The one exchange of the sharded step: all-gather of every rank's [K, M] table of local sums of
    squares (float64).  Returns the tables of all ranks in rank order, shape [world, K, M], on the
    device of ``local``.  Works with any torch.distributed backend (NCCL on GPUs, gloo on CPU); on
    a GPU the collective is ordered against torch's current stream."""
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    K, M = local.shape
    gathered = torch.empty(world * K, M, dtype=local.dtype, device=local.device)      # rank-major
    dist.all_gather_into_tensor(gathered, local.contiguous(), group=group)
    return gathered.view(world, K, M)


def _stream_context(stream):
    """Makes ``stream`` (None, a torch.cuda.Stream or a raw cudaStream_t) torch's current stream, so
    that allocations, the library's kernels and the collective are all ordered on it."""
    import contextlib

    import torch
    if stream is None:
        return contextlib.nullcontext()
    if not isinstance(stream, torch.cuda.Stream):
        stream = torch.cuda.ExternalStream(int(stream))
    return torch.cuda.stream(stream)


def sharded_step(variant, params, grads, pull, local_offsets, center_out=None, *, group=None, stream=None):
    """One averaging step on this rank's element range.

    params, grads: this rank's slices of the M replicas (device float32, bfloat16 or float16 tensors of
    j1-j0 elements, all of one type);
    local_offsets: local_layer_table(...) of the range.  Collective: every rank of `group` must call it.
    Everything (the two library calls and the all-gather between them) is enqueued on ``stream``
    (default: torch's current stream).
    """
    import torch
    import torch.distributed as dist

    world = dist.get_world_size(group)
    K, M = len(local_offsets) - 1, len(params)
    with _stream_context(stream):
        local = torch.empty(K, M, dtype=torch.float64, device=params[0].device)
        binding.grawa_layer_sumsq_typed(grads, local_offsets, local)          # storage type taken from the tensors
        gathered = exchange_layer_sums(local, group)
        binding.grawa_step_from_layer_sums_typed(variant, params, gathered, world, pull, local_offsets, center_out)
